// extern "C" boundary of libfbq: argument validation, kernel selection,
// per-stream scratch space, launch bookkeeping.  Declarations and the contract
// of every entry point are in include/fbq.h.
#include <atomic>
#include <cstring>
#include <map>
#include <mutex>
#include <utility>

#include "fbq_common.cuh"

namespace fbq {
void decode_set_test_switch(int t_late);
void decode_set_t_wait(int on);
void prefill_set_pair(int on);
void prefill_set_split(int mode);
void prefill_set_pdl(int on);
void prefill_set_test(int skip_flag, int flag_polls);

namespace {

std::mutex g_mu;
std::map<std::pair<int, cudaStream_t>, Workspace> g_ws;
std::atomic<long long> g_launches{0};

struct Options {
    int force_kernel = -1;
    DecodeTuning decode;
    GemvTuning gemv;
    int use_gemv = 1;
    int decode_t_late = 0;
    int decode_t_wait = 1;
    int batch_ctas = 400;
    int batch_single = 1;
    int prefill_pair = 0;
    int prefill_split = 2;
    int hostio_direct_y = 1;
    int test_prefill_skip_flag = 0, prefill_flag_polls = 0;
    int decode_trace = 0;
} g_opt;
constexpr size_t kTraceBytes = 512 * 18 * 16 * 8;   // 512 CTAs x up to 18 warps x 16 marks

bool misaligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

// The host-buffer entry points write a small y straight into the caller's buffer when that is pinned host memory
// which the GPU can address (unified addressing): the kernel's stores cross the bus instead of a copy that would
// have to be queued behind the kernel.  Returns the buffer's device alias, or nullptr (pageable memory, unaligned,
// large, switched off): then y goes through the stream's staging buffer and a copy.
void *direct_y_alias(void *y_host, size_t bytes)
{
    if (!g_opt.hostio_direct_y || bytes > (256u << 10)) return nullptr;
    cudaPointerAttributes at{};
    if (cudaPointerGetAttributes(&at, y_host) != cudaSuccess) {
        (void)cudaGetLastError();
        return nullptr;
    }
    if (at.type != cudaMemoryTypeHost || !at.devicePointer || misaligned16(at.devicePointer)) return nullptr;
    return at.devicePointer;
}

bool well_formed(int M, int N, int K, int group, int bits, int rank)
{
    if (M < 0 || N < 1 || K < 1 || group < 1 || rank < 0) return false;
    if (bits != 3 && bits != 4) return false;
    const int unit = (bits == 4) ? 8 : 32;
    if (group % unit != 0 || K % group != 0) return false;
    return true;
}

int select_kernel(int M, int N, int K, int group, int bits, int rank, bool bf16)
{
    if (!well_formed(M, N, K, group, bits, rank)) return FBQ_KERNEL_NONE;
    LinearArgs a{};
    a.M = M; a.N = N; a.K = K; a.group = group; a.bits = bits; a.rank = rank; a.bf16 = bf16;
    const bool fast_group = (group == kGroupFast) && rank % 8 == 0 && rank <= kMaxRank;
    const bool decode_ok = fast_group && M >= 1 && M <= kDecodeMaxM;
    const bool prefill_ok = fast_group && M >= 1 && prefill_supported(a);
    if (g_opt.force_kernel == FBQ_KERNEL_GENERIC) return FBQ_KERNEL_GENERIC;
    if (g_opt.force_kernel == FBQ_KERNEL_DECODE && decode_ok) return FBQ_KERNEL_DECODE;
    if (g_opt.force_kernel == FBQ_KERNEL_PREFILL && prefill_ok) return FBQ_KERNEL_PREFILL;
    if (g_opt.force_kernel >= 0) return FBQ_KERNEL_GENERIC;
    // Measured on B200 (7B layer, INT4, one stream in layer order, us per layer step, rank 16 / 64 / 128 / 0):
    //   streaming decode kernel   M = 4: 84 / 87 / 101 / 74    M = 8: 107 / 112 / 144 / 91   M = 12: 142 / 156 / 202 / 114   M = 16: 160 / 176 / 236 / 125
    //   tensor-core kernel        M = 4: 213                   M = 8: 211                    M = 12: 192 / 207 / 213 / 178   M = 16: 176 / 197 / 201 / 166
    //                             (K split whenever tiles are few, the default; 227 - 257 with the split only for K >= 8192)
    //   the other decode kernel   M = 4: 129                   M = 8: 258                    M = 16: 3204
    // per shape at rank 128 (us per launch, 4096 -> 4096 / 4096 -> 11008 / 11008 -> 4096): streaming M = 12: 21.7 / 29.6 / 58.6,
    // M = 16: 24.9 / 34.0 / 68.9; tensor-core M = 12: 23.6 / 40.1 / 35.1, M = 16: 23.7 / 35.4 / 35.3;
    // and on the 13B layer (K = 5120 / 13824; rank 64 / 0): streaming M = 8: 150 / 125, M = 12: 208 / 163, M = 16: 411 / 307;
    // tensor-core M = 8: 256 / 232, M = 12: 258 / 231, M = 16: 234 / 206.  Above eight tokens the streaming kernel
    // pays only while x of all K fits its shared memory (one K slice: M * K * 2 bytes up to 136 KB), so where its
    // domain allows it takes M <= 8 for every shape, and M <= 16 for the shapes it does not have to slice.
    // Outside that domain the other decode kernel keeps its own crossover: up to M = 4 it gets t from CTAs at the
    // head of its grid and wins at every rank up to 128; at M = 5 and 6 every CTA contributes to t and the tiles
    // wait for it, work that grows with M * rank, so M * rank above 128 goes to the tensor-core kernel.
    const bool streaming = g_opt.use_gemv != 0 && decode_ok && gemv_supported(a);
    const bool decode_pays = streaming ? (M <= 8 || gemv_k_slices(M, K) == 1)
                                       : (M <= kDecodePreferM && (M <= 4 ? rank <= 128 : M * rank <= 128));
    if (decode_ok && (decode_pays || !prefill_ok)) return FBQ_KERNEL_DECODE;
    if (prefill_ok) return FBQ_KERNEL_PREFILL;
    return FBQ_KERNEL_GENERIC;
}

// Grows a device buffer; zero-fills it on `s` (the invariants of the decode
// kernel's scratch space start from zero).  The old buffer is released only
// after the stream has drained.
template <typename P>
cudaError_t grow(P *&ptr, size_t &have, size_t need, size_t elem, cudaStream_t s)
{
    if (need <= have) return cudaSuccess;
    cudaError_t e;
    // Allocating (and, for a buffer that exists, synchronising and freeing) is illegal while `s` is being
    // captured into a graph, and a graph captured earlier would keep the old pointers: refuse instead.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(s, &cap) == cudaSuccess && cap != cudaStreamCaptureStatusNone) return cudaErrorStreamCaptureUnsupported;
    if (ptr) {
        if ((e = cudaStreamSynchronize(s)) != cudaSuccess) return e;
        if ((e = cudaFree(ptr)) != cudaSuccess) return e;
        ptr = nullptr;
        have = 0;
    }
    void *q = nullptr;
    if ((e = cudaMalloc(&q, need * elem)) != cudaSuccess) return e;
    if ((e = cudaMemsetAsync(q, 0, need * elem, s)) != cudaSuccess) {
        cudaFree(q);
        return e;
    }
    ptr = static_cast<P *>(q);
    have = need;
    return cudaSuccess;
}

Workspace *workspace_for(cudaStream_t s)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    std::lock_guard<std::mutex> lk(g_mu);
    return &g_ws[std::make_pair(dev, s)];
}

int grow_status(cudaError_t e) { return e == cudaErrorStreamCaptureUnsupported ? FBQ_ERR_UNSUPPORTED : FBQ_ERR_CUDA; }

// decode_ctas > 0 overrides the decode kernel's grid-size bound for this call.
int run_linear(const LinearArgs &a, cudaStream_t s, int decode_ctas = 0)
{
    DecodeTuning tune = g_opt.decode;
    if (decode_ctas > 0) tune.max_ctas = decode_ctas;
    if (!well_formed(a.M, a.N, a.K, a.group, a.bits, a.rank)) return FBQ_ERR_BADARG;
    if (a.M == 0) return FBQ_OK;
    if (!a.x || !a.qw || !a.scales || !a.zeros || !a.y) return FBQ_ERR_BADARG;
    if (a.rank > 0 && (!a.A || !a.B)) return FBQ_ERR_BADARG;
    if (misaligned16(a.x) || misaligned16(a.qw) || misaligned16(a.y) || (a.rank > 0 && (misaligned16(a.A) || misaligned16(a.B))))
        return FBQ_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(a.scales) & 1u) || (reinterpret_cast<uintptr_t>(a.zeros) & 1u)) return FBQ_ERR_ALIGN;

    Workspace *ws = workspace_for(s);
    if (!ws) return FBQ_ERR_CUDA;
    int kernel = select_kernel(a.M, a.N, a.K, a.group, a.bits, a.rank, a.bf16);
    if (kernel == FBQ_KERNEL_NONE) return FBQ_ERR_UNSUPPORTED;
    int launches = 0;
    cudaError_t e = cudaSuccess;

    if (kernel == FBQ_KERNEL_DECODE && g_opt.use_gemv && gemv_supported(a)) {
        GemvTuning gt = g_opt.gemv;
        gt.pdl = g_opt.decode.pdl;
        if (tune.max_ctas > 0) gt.max_ctas = tune.max_ctas;
        size_t pf = 0, partf = 0;
        int nc = 0;
        gemv_workspace_need(a, gt, &pf, &nc, &partf);
        size_t have_c = (size_t)ws->n_counters;
        if ((e = grow(ws->tslots, ws->tslots_floats, pf, sizeof(float), s)) != cudaSuccess) return grow_status(e);
        if (partf > 0 && (e = grow(ws->partial, ws->partial_floats, partf, sizeof(float), s)) != cudaSuccess) return grow_status(e);
        if ((e = grow(ws->counters, have_c, (size_t)nc, sizeof(int), s)) != cudaSuccess) return grow_status(e);
        ws->n_counters = (int)have_c;
        if (g_opt.decode_trace && !ws->trace) {
            if (cudaMalloc(&ws->trace, kTraceBytes) != cudaSuccess) return FBQ_ERR_CUDA;
            cudaMemset(ws->trace, 0, kTraceBytes);
        }
        e = launch_gemv(a, *ws, gt, s, &launches);
        if (e == cudaSuccess) {
            g_launches += launches;
            return FBQ_OK;
        }
        if (e != cudaErrorInvalidConfiguration) return FBQ_ERR_CUDA;
        (void)cudaGetLastError();                 // no plan fits: the other decode kernel
    }
    if (kernel == FBQ_KERNEL_DECODE) {
        size_t pf = 0;
        int nc = 0;
        decode_workspace_need(a, tune, &pf, &nc);
        size_t have_c = (size_t)ws->n_counters;
        if ((e = grow(ws->partial, ws->partial_floats, pf, sizeof(float), s)) != cudaSuccess) return grow_status(e);
        if ((e = grow(ws->t, ws->t_floats, (size_t)kDecodeMaxM * kMaxRank, sizeof(float), s)) != cudaSuccess) return grow_status(e);
        if ((e = grow(ws->counters, have_c, (size_t)nc, sizeof(int), s)) != cudaSuccess) return grow_status(e);
        ws->n_counters = (int)have_c;
        if (g_opt.decode_trace && !ws->trace) {
            if (cudaMalloc(&ws->trace, kTraceBytes) != cudaSuccess) return FBQ_ERR_CUDA;
        }
        if (ws->trace) {
            if (!g_opt.decode_trace) {
                cudaStreamSynchronize(s);
                cudaFree(ws->trace);
                ws->trace = nullptr;
            }
        }
        e = launch_decode(a, *ws, tune, s, &launches);
        if (e == cudaErrorInvalidConfiguration) {
            (void)cudaGetLastError();
            kernel = FBQ_KERNEL_GENERIC;          // plan does not fit shared memory
        } else if (e != cudaSuccess) {
            return FBQ_ERR_CUDA;
        }
    }
    if (kernel == FBQ_KERNEL_PREFILL) {
        size_t have_c = (size_t)ws->n_counters, need_t = 0, need_p = 0;
        int need_c = 0;
        prefill_workspace_need(a, &need_c, &need_t, &need_p);
        if ((e = grow(ws->counters, have_c, (size_t)need_c, sizeof(int), s)) != cudaSuccess) return grow_status(e);
        ws->n_counters = (int)have_c;
        if (need_t > 0 && (e = grow(ws->t_gen, ws->t_gen_floats, need_t, sizeof(float), s)) != cudaSuccess) return grow_status(e);
        if (need_p > 0 && (e = grow(ws->partial, ws->partial_floats, need_p, sizeof(float), s)) != cudaSuccess) return grow_status(e);
        e = launch_prefill(a, *ws, s, &launches);
        if (e == cudaErrorInvalidConfiguration) {
            (void)cudaGetLastError();
            kernel = FBQ_KERNEL_GENERIC;
        } else if (e != cudaSuccess) {
            return FBQ_ERR_CUDA;
        }
    }
    if (kernel == FBQ_KERNEL_GENERIC) {
        if (a.rank > 0 &&
            (e = grow(ws->t_gen, ws->t_gen_floats, (size_t)a.M * a.rank, sizeof(float), s)) != cudaSuccess)
            return FBQ_ERR_CUDA;
        if ((e = launch_generic(a, *ws, s, &launches)) != cudaSuccess) return FBQ_ERR_CUDA;
    }
    g_launches += launches;
    return FBQ_OK;
}

int *option_slot(const char *name)
{
    if (!name) return nullptr;
    if (!strcmp(name, "force_kernel")) return &g_opt.force_kernel;
    if (!strcmp(name, "gemv")) return &g_opt.use_gemv;
    if (!strcmp(name, "gemv_ctas")) return &g_opt.gemv.max_ctas;
    if (!strcmp(name, "t_poll_limit")) return &g_opt.gemv.poll_limit;
    if (!strcmp(name, "test_skip_t_arrive")) return &g_opt.gemv.test_skip_arrive;
    if (!strcmp(name, "decode_sk")) return &g_opt.decode.sk;
    if (!strcmp(name, "decode_chunk")) return &g_opt.decode.chunk;
    if (!strcmp(name, "decode_depth")) return &g_opt.decode.depth;
    if (!strcmp(name, "decode_ctas")) return &g_opt.decode.max_ctas;
    if (!strcmp(name, "decode_i8")) return &g_opt.decode.i8;
    if (!strcmp(name, "decode_t_ctas")) return &g_opt.decode.t_ctas;
    if (!strcmp(name, "decode_t_wait")) return &g_opt.decode_t_wait;
    if (!strcmp(name, "pdl")) return &g_opt.decode.pdl;
    if (!strcmp(name, "decode_t_late")) return &g_opt.decode_t_late;
    if (!strcmp(name, "batch_ctas")) return &g_opt.batch_ctas;
    if (!strcmp(name, "batch_single")) return &g_opt.batch_single;
    if (!strcmp(name, "prefill_pair")) return &g_opt.prefill_pair;
    if (!strcmp(name, "prefill_split")) return &g_opt.prefill_split;
    if (!strcmp(name, "hostio_direct_y")) return &g_opt.hostio_direct_y;
    if (!strcmp(name, "test_prefill_skip_flag")) return &g_opt.test_prefill_skip_flag;
    if (!strcmp(name, "prefill_flag_polls")) return &g_opt.prefill_flag_polls;
    if (!strcmp(name, "decode_trace")) return &g_opt.decode_trace;
    return nullptr;
}

}  // namespace

void count_launches(int n) { g_launches += n; }

int noalloc_poll_status(int dev);      // fbq_noalloc.cu

// For the no-allocation entry point: the process-wide switches applied, and the decode tuning with
// everything that sizes scratch left automatic.
DecodeTuning decode_tuning_for_noalloc()
{
    decode_set_test_switch(g_opt.decode_t_late);
    decode_set_t_wait(g_opt.decode_t_wait);
    DecodeTuning t = g_opt.decode;
    t.max_ctas = 0;
    t.sk = 0;
    return t;
}

}  // namespace fbq

using namespace fbq;

extern "C" {

size_t fbq_packed_words(int N, int K, int bits)
{
    if (N < 1 || K < 1) return 0;
    if (bits == 4 && K % 8 == 0) return (size_t)N * K / 8;
    if (bits == 3 && K % 32 == 0) return (size_t)N * K / 32 * 3;
    return 0;
}

static int pack_common(const uint8_t *codes, uint32_t *qweight, int N, int K, int bits, void *stream)
{
    if (!codes || !qweight || fbq_packed_words(N, K, bits) == 0) return FBQ_ERR_BADARG;
    if (misaligned16(codes) || misaligned16(qweight)) return FBQ_ERR_ALIGN;
    if (launch_pack(codes, qweight, N, K, bits, static_cast<cudaStream_t>(stream)) != cudaSuccess) return FBQ_ERR_CUDA;
    ++g_launches;
    return FBQ_OK;
}

int fbq_pack_int4(const uint8_t *codes, uint32_t *qweight, int N, int K, void *stream)
{
    return pack_common(codes, qweight, N, K, 4, stream);
}

int fbq_pack_int3(const uint8_t *codes, uint32_t *qweight, int N, int K, void *stream)
{
    return pack_common(codes, qweight, N, K, 3, stream);
}

int fbq_unpack(const uint32_t *qweight, uint8_t *codes, int N, int K, int bits, void *stream)
{
    if (!codes || !qweight || fbq_packed_words(N, K, bits) == 0) return FBQ_ERR_BADARG;
    if (misaligned16(codes) || misaligned16(qweight)) return FBQ_ERR_ALIGN;
    if (launch_unpack(qweight, codes, N, K, bits, static_cast<cudaStream_t>(stream)) != cudaSuccess) return FBQ_ERR_CUDA;
    ++g_launches;
    return FBQ_OK;
}

int fbq_dequant(const uint32_t *qweight, const uint16_t *scales, const uint16_t *zeros, float *W, int N, int K,
                int group, int bits, void *stream)
{
    if (!qweight || !scales || !zeros || !W) return FBQ_ERR_BADARG;
    if (!well_formed(1, N, K, group, bits, 0)) return FBQ_ERR_BADARG;
    if (misaligned16(qweight) || misaligned16(W)) return FBQ_ERR_ALIGN;
    if (launch_dequant(qweight, reinterpret_cast<const __half *>(scales), reinterpret_cast<const __half *>(zeros), W, N,
                       K, group, bits, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return FBQ_ERR_CUDA;
    ++g_launches;
    return FBQ_OK;
}

int fbq_quantize_feedback(const float *W, const void *A, const void *B, uint8_t *codes, void *scales, void *zeros,
                          float *WF, int N, int K, int group, int bits, int rank, int act_is_bf16, void *stream)
{
    if (N < 1 || K < 1 || group < 1 || group > 1024 || K % group != 0 || K / group > 65535 || rank < 0) return FBQ_ERR_BADARG;
    if (bits != 3 && bits != 4) return FBQ_ERR_BADARG;
    if (!W || !codes || !scales || !zeros || (rank > 0 && (!A || !B))) return FBQ_ERR_BADARG;
    if ((reinterpret_cast<uintptr_t>(W) & 3u) || (WF && (reinterpret_cast<uintptr_t>(WF) & 3u)) ||
        (reinterpret_cast<uintptr_t>(scales) & 1u) || (reinterpret_cast<uintptr_t>(zeros) & 1u) ||
        (rank > 0 && ((reinterpret_cast<uintptr_t>(A) & 1u) || (reinterpret_cast<uintptr_t>(B) & 1u))))
        return FBQ_ERR_ALIGN;
    if (launch_quantize_feedback(W, A, B, codes, static_cast<__half *>(scales), static_cast<__half *>(zeros), WF, nullptr, N, K,
                                 group, bits, rank, act_is_bf16 ? 1 : 0, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return FBQ_ERR_CUDA;
    ++g_launches;
    return FBQ_OK;
}

size_t fbq_reconstruct_workspace_floats(int N, int K, int rank)
{
    if (N < 1 || K < 1 || rank < 1) return 0;
    return reconstruct_workspace_floats(N, K, rank);
}

int fbq_gram(const float *X, float *H, int T, int K, void *stream)
{
    if (!X || !H || T < 1 || K < 1) return FBQ_ERR_BADARG;
    const int rc = run_gram(X, H, T, K, static_cast<cudaStream_t>(stream));
    if (rc == FBQ_OK) ++g_launches;
    return rc;
}

int fbq_reconstruct_step(const float *W, const float *H, float *A, float *B, float lr, float *loss, float *workspace, int N,
                         int K, int group, int bits, int rank, void *stream)
{
    if (N < 1 || K < 1 || rank < 1 || group < 1 || group > 1024 || K % group != 0 || K / group > 65535) return FBQ_ERR_BADARG;
    if (bits != 3 && bits != 4) return FBQ_ERR_BADARG;
    if (!W || !H || !A || !B || !workspace) return FBQ_ERR_BADARG;
    const int rc = run_reconstruct_step(W, H, A, B, lr, loss, workspace, N, K, group, bits, rank, static_cast<cudaStream_t>(stream));
    if (rc == FBQ_OK) g_launches += loss ? 8 : 6;       // quantiser, three GEMMs, (two-stage reduction), two updates
    return rc;
}

// Hands the process-wide switches to the kernel files before a launch.
static void apply_kernel_options()
{
    decode_set_test_switch(g_opt.decode_t_late);
    decode_set_t_wait(g_opt.decode_t_wait);
    prefill_set_pair(g_opt.prefill_pair);
    prefill_set_split(g_opt.prefill_split);
    prefill_set_pdl(g_opt.decode.pdl);
    prefill_set_test(g_opt.test_prefill_skip_flag, g_opt.prefill_flag_polls);
}

static int linear_common(const void *x, const uint32_t *qweight, const void *scales, const void *zeros, const void *A,
                         const void *B, void *y, int M, int N, int K, int group, int bits, int rank, bool bf16,
                         void *stream)
{
    LinearArgs a{};
    a.x = x; a.qw = qweight;
    a.scales = static_cast<const __half *>(scales);
    a.zeros = static_cast<const __half *>(zeros);
    a.A = rank > 0 ? A : nullptr;
    a.B = rank > 0 ? B : nullptr;
    a.y = y;
    a.M = M; a.N = N; a.K = K; a.group = group; a.bits = bits; a.rank = rank; a.bf16 = bf16;
    apply_kernel_options();
    return run_linear(a, static_cast<cudaStream_t>(stream));
}

int fbq_linear(const void *x, const uint32_t *qweight, const void *scales, const void *zeros, const void *A,
               const void *B, void *y, int M, int N, int K, int group, int bits, int rank, void *stream)
{
    return linear_common(x, qweight, scales, zeros, A, B, y, M, N, K, group, bits, rank, false, stream);
}

int fbq_linear_bf16(const void *x, const uint32_t *qweight, const void *scales, const void *zeros, const void *A,
                    const void *B, void *y, int M, int N, int K, int group, int bits, int rank, void *stream)
{
    return linear_common(x, qweight, scales, zeros, A, B, y, M, N, K, group, bits, rank, true, stream);
}

// Side streams and events of fbq_linear_batch, per device, created on first use and kept.
struct BatchLanes {
    cudaStream_t side[FBQ_BATCH_MAX] = {};
    cudaEvent_t fork = nullptr, join[FBQ_BATCH_MAX] = {};
    int n = 0;
};
static std::map<int, BatchLanes> g_lanes;

static BatchLanes *lanes_for(int want)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    std::lock_guard<std::mutex> lk(g_mu);
    BatchLanes &b = g_lanes[dev];
    if (!b.fork && cudaEventCreateWithFlags(&b.fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    while (b.n < want) {
        if (cudaStreamCreateWithFlags(&b.side[b.n], cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        if (cudaEventCreateWithFlags(&b.join[b.n], cudaEventDisableTiming) != cudaSuccess) return nullptr;
        ++b.n;
    }
    return &b;
}

static int linear_batch_common(const fbq_problem *problems, int count, int M, int group, int bits, int rank, int act_is_bf16,
                               void *stream, bool host_io)
{
    if (count < 0 || count > FBQ_BATCH_MAX || (count > 0 && !problems)) return FBQ_ERR_BADARG;
    if (count == 0) return FBQ_OK;
    cudaStream_t main = static_cast<cudaStream_t>(stream);
    apply_kernel_options();
    LinearArgs a[FBQ_BATCH_MAX];
    bool all_decode = count > 1;
    double total_cost = 0.0;
    for (int i = 0; i < count; ++i) {
        const fbq_problem &q = problems[i];
        a[i] = LinearArgs{};
        a[i].x = q.x; a[i].qw = q.qweight;
        a[i].scales = static_cast<const __half *>(q.scales);
        a[i].zeros = static_cast<const __half *>(q.zeros);
        a[i].A = rank > 0 ? q.A : nullptr;
        a[i].B = rank > 0 ? q.B : nullptr;
        a[i].y = q.y;
        a[i].M = M; a[i].N = q.N; a[i].K = q.K; a[i].group = group; a[i].bits = bits; a[i].rank = rank;
        a[i].bf16 = act_is_bf16 != 0;
        if (!well_formed(M, q.N, q.K, group, bits, rank)) return FBQ_ERR_BADARG;
        all_decode = all_decode && select_kernel(M, q.N, q.K, group, bits, rank, a[i].bf16) == FBQ_KERNEL_DECODE;
        total_cost += (double)q.N * q.K;
    }
    // With host_io, x and y of every problem are host buffers: x is copied to, and y back from,
    // staging buffers kept per stream, on the stream the problem runs on.
    auto stage_in = [&](LinearArgs &la, cudaStream_t st) -> int {
        if (!host_io) return FBQ_OK;
        Workspace *ws = workspace_for(st);
        if (!ws || !la.x || !la.y) return ws ? FBQ_ERR_BADARG : FBQ_ERR_CUDA;
        const size_t xb = (size_t)M * la.K * 2, yb = (size_t)M * la.N * 2;
        char *sx = static_cast<char *>(ws->stage_x), *sy = static_cast<char *>(ws->stage_y);
        if (grow(sx, ws->stage_x_bytes, xb, 1, st) != cudaSuccess) return FBQ_ERR_CUDA;
        ws->stage_x = sx;
        if (cudaMemcpyAsync(sx, la.x, xb, cudaMemcpyHostToDevice, st) != cudaSuccess) return FBQ_ERR_CUDA;
        la.x = sx;
        if (void *alias = direct_y_alias(la.y, yb)) {
            la.y = alias;                             // the kernel writes the caller's buffer itself
            return FBQ_OK;
        }
        if (grow(sy, ws->stage_y_bytes, yb, 1, st) != cudaSuccess) return FBQ_ERR_CUDA;
        ws->stage_y = sy;
        la.y = sy;
        return FBQ_OK;
    };
    auto stage_out = [&](const LinearArgs &la, void *y_host, cudaStream_t st) -> int {
        if (!host_io) return FBQ_OK;
        Workspace *ws = workspace_for(st);
        if (!ws || la.y != ws->stage_y) return FBQ_OK;      // written in place
        return cudaMemcpyAsync(y_host, la.y, (size_t)M * la.N * 2, cudaMemcpyDeviceToHost, st) == cudaSuccess ? FBQ_OK : FBQ_ERR_CUDA;
    };
    if (!all_decode) {
        // one after the other on the caller's stream (prefill-sized problems fill the GPU by themselves)
        for (int i = 0; i < count; ++i) {
            int rc = stage_in(a[i], main);
            if (rc == FBQ_OK) rc = run_linear(a[i], main);
            if (rc == FBQ_OK) rc = stage_out(a[i], problems[i].y, main);
            if (rc != FBQ_OK) return rc;
        }
        return FBQ_OK;
    }
    // Decode-sized problems: all at once, grids in proportion to the problems' share of the codes so
    // that the CTAs of the whole batch are resident together and finish together.
    int ctas[FBQ_BATCH_MAX];
    for (int i = 0; i < count; ++i)
        ctas[i] = std::max(8, (int)(g_opt.batch_ctas * ((double)a[i].N * a[i].K / total_cost) + 0.5));
    // Problems in the streaming kernel's domain run as one launch each on the side streams (the same kernel, hence
    // the same sums, as fbq_linear); the single launch over a problem list is the other decode kernel's.
    bool all_gemv = g_opt.use_gemv != 0;
    for (int i = 0; i < count; ++i) all_gemv = all_gemv && gemv_supported(a[i]);
    if (g_opt.batch_single && !host_io && count <= decode_batch_max() && !all_gemv) {
        // One launch: the decode kernel over a problem list, on the caller's stream.  (With host
        // buffers the per-problem streams below are faster: their small copies overlap.)
        for (int i = 0; i < count; ++i) {
            if (!a[i].x || !a[i].qw || !a[i].scales || !a[i].zeros || !a[i].y || (rank > 0 && (!a[i].A || !a[i].B)))
                return FBQ_ERR_BADARG;
            if (misaligned16(a[i].qw) || (rank > 0 && (misaligned16(a[i].A) || misaligned16(a[i].B))) || misaligned16(a[i].x) ||
                misaligned16(a[i].y))
                return FBQ_ERR_ALIGN;
        }
        Workspace *ws = workspace_for(main);
        if (!ws) return FBQ_ERR_CUDA;
        size_t pf = 0, tf = 0;
        int nc = 0;
        if (decode_batch_need(a, count, ctas, g_opt.decode, &pf, &tf, &nc)) {
            size_t have_c = (size_t)ws->n_counters;
            if (grow(ws->partial, ws->partial_floats, pf, sizeof(float), main) != cudaSuccess) return FBQ_ERR_CUDA;
            if (grow(ws->t, ws->t_floats, tf, sizeof(float), main) != cudaSuccess) return FBQ_ERR_CUDA;
            if (grow(ws->counters, have_c, (size_t)nc, sizeof(int), main) != cudaSuccess) return FBQ_ERR_CUDA;
            ws->n_counters = (int)have_c;
            int launches = 0;
            const cudaError_t e = launch_decode_batch(a, count, ctas, *ws, g_opt.decode, main, &launches);
            if (e != cudaSuccess) return FBQ_ERR_CUDA;
            g_launches += launches;
            return FBQ_OK;
        }
        // a problem has no decode plan: fall through to one launch per problem
    }
    // One launch per problem: problem i runs on side stream i, forked from and joined to the caller's
    // stream by events.
    BatchLanes *lanes = lanes_for(count);
    if (!lanes) return FBQ_ERR_CUDA;
    if (cudaEventRecord(lanes->fork, main) != cudaSuccess) return FBQ_ERR_CUDA;
    int rc = FBQ_OK;
    int forked = 0;
    for (int i = 0; i < count; ++i) {
        if (cudaStreamWaitEvent(lanes->side[i], lanes->fork, 0) != cudaSuccess) { rc = FBQ_ERR_CUDA; break; }
        ++forked;
        rc = stage_in(a[i], lanes->side[i]);
        if (rc == FBQ_OK) rc = run_linear(a[i], lanes->side[i], ctas[i]);
        if (rc == FBQ_OK) rc = stage_out(a[i], problems[i].y, lanes->side[i]);
        if (rc != FBQ_OK) break;
    }
    for (int i = 0; i < forked; ++i) {              // always rejoin what was forked (also under stream capture)
        if (cudaEventRecord(lanes->join[i], lanes->side[i]) != cudaSuccess ||
            cudaStreamWaitEvent(main, lanes->join[i], 0) != cudaSuccess)
            rc = (rc == FBQ_OK) ? FBQ_ERR_CUDA : rc;
    }
    return rc;
}

int fbq_linear_batch(const fbq_problem *problems, int count, int M, int group, int bits, int rank, int act_is_bf16,
                     void *stream)
{
    return linear_batch_common(problems, count, M, group, bits, rank, act_is_bf16, stream, false);
}

int fbq_linear_batch_hostio(const fbq_problem *problems, int count, int M, int group, int bits, int rank, int act_is_bf16,
                            void *stream)
{
    return linear_batch_common(problems, count, M, group, bits, rank, act_is_bf16, stream, true);
}

int fbq_linear_hostio(const void *x_host, const uint32_t *qweight, const void *scales, const void *zeros,
                      const void *A, const void *B, void *y_host, int M, int N, int K, int group, int bits, int rank,
                      int act_is_bf16, void *stream)
{
    if (!well_formed(M, N, K, group, bits, rank)) return FBQ_ERR_BADARG;
    if (M == 0) return FBQ_OK;
    if (!x_host || !y_host) return FBQ_ERR_BADARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Workspace *ws = workspace_for(s);
    if (!ws) return FBQ_ERR_CUDA;
    const size_t xb = (size_t)M * K * 2, yb = (size_t)M * N * 2;
    char *sx = static_cast<char *>(ws->stage_x), *sy = static_cast<char *>(ws->stage_y);
    if (grow(sx, ws->stage_x_bytes, xb, 1, s) != cudaSuccess) return FBQ_ERR_CUDA;
    ws->stage_x = sx;
    if (cudaMemcpyAsync(sx, x_host, xb, cudaMemcpyHostToDevice, s) != cudaSuccess) return FBQ_ERR_CUDA;
    if (void *alias = direct_y_alias(y_host, yb))       // the kernel writes the caller's buffer itself
        return linear_common(sx, qweight, scales, zeros, A, B, alias, M, N, K, group, bits, rank, act_is_bf16 != 0, stream);
    if (grow(sy, ws->stage_y_bytes, yb, 1, s) != cudaSuccess) return FBQ_ERR_CUDA;
    ws->stage_y = sy;
    const int rc = linear_common(sx, qweight, scales, zeros, A, B, sy, M, N, K, group, bits, rank, act_is_bf16 != 0, stream);
    if (rc != FBQ_OK) return rc;
    if (cudaMemcpyAsync(y_host, sy, yb, cudaMemcpyDeviceToHost, s) != cudaSuccess) return FBQ_ERR_CUDA;
    return FBQ_OK;
}

int fbq_sub_branch_unfused(const void *x, const void *A, const void *B, void *y, int M, int N, int K, int rank, int act_is_bf16,
                            void *stream)
{
    if (M < 0 || N < 1 || K < 1 || rank < 1) return FBQ_ERR_BADARG;
    if (M == 0) return FBQ_OK;
    if (!x || !A || !B || !y) return FBQ_ERR_BADARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Workspace *ws = workspace_for(s);
    if (!ws) return FBQ_ERR_CUDA;
    cudaError_t e;
    if ((e = grow(ws->t_gen, ws->t_gen_floats, (size_t)M * rank + ((size_t)M * N + 1) / 2 + 4, sizeof(float), s)) != cudaSuccess)
        return grow_status(e);
    int launches = 0;
    if (launch_sub_branch_unfused(x, A, B, y, M, N, K, rank, act_is_bf16 != 0, *ws, s, &launches) != cudaSuccess) return FBQ_ERR_CUDA;
    g_launches += launches;
    return FBQ_OK;
}

int fbq_select_kernel(int M, int N, int K, int group, int bits, int rank, int act_is_bf16)
{
    return select_kernel(M, N, K, group, bits, rank, act_is_bf16 != 0);
}

int fbq_set_option(const char *name, int value)
{
    int *slot = option_slot(name);
    if (!slot) return FBQ_ERR_BADARG;
    *slot = value;
    return FBQ_OK;
}

int fbq_get_option(const char *name, int *value)
{
    int *slot = option_slot(name);
    if (!slot || !value) return FBQ_ERR_BADARG;
    *value = *slot;
    return FBQ_OK;
}

long long fbq_launch_count(void) { return g_launches.load(); }

int fbq_poll_status(void *stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(s) != cudaSuccess) return FBQ_ERR_CUDA;
    Workspace *ws = workspace_for(s);
    if (!ws) return FBQ_ERR_CUDA;
    // the fixed scratch array of fbq_linear_noalloc has a status word of its own (shared by all streams)
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return FBQ_ERR_CUDA;
    const int fixed = noalloc_poll_status(dev);
    if (fixed != FBQ_OK) return fixed;
    if (!ws->counters) return FBQ_OK;
    int st = 0;
    if (cudaMemcpy(&st, ws->counters + kCtrStatus, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return FBQ_ERR_CUDA;
    if (st != 0) {
        // a kernel gave up half way: its bookkeeping is unfinished, start from a clean slate
        cudaMemset(ws->counters, 0, sizeof(int) * (size_t)ws->n_counters);
        if (ws->t) cudaMemset(ws->t, 0, sizeof(float) * ws->t_floats);
        if (ws->tslots) cudaMemset(ws->tslots, 0, sizeof(float) * ws->tslots_floats);
    }
    return st;
}

int fbq_debug_read_trace(void *stream, void *host_buf, size_t bytes)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(s) != cudaSuccess) return FBQ_ERR_CUDA;
    Workspace *ws = workspace_for(s);
    if (!ws || !ws->trace || !host_buf || bytes > kTraceBytes) return FBQ_ERR_BADARG;
    return cudaMemcpy(host_buf, ws->trace, bytes, cudaMemcpyDeviceToHost) == cudaSuccess ? FBQ_OK : FBQ_ERR_CUDA;
}

int fbq_release_workspaces(void)
{
    if (cudaDeviceSynchronize() != cudaSuccess) return FBQ_ERR_CUDA;
    std::lock_guard<std::mutex> lk(g_mu);
    for (auto &kv : g_ws) {
        Workspace &w = kv.second;
        cudaFree(w.partial);
        cudaFree(w.t);
        cudaFree(w.t_gen);
        cudaFree(w.tslots);
        cudaFree(w.counters);
        cudaFree(w.trace);
        cudaFree(w.stage_x);
        cudaFree(w.stage_y);
    }
    g_ws.clear();
    return FBQ_OK;
}

const char *fbq_status_string(int status)
{
    switch (status) {
    case FBQ_OK: return "ok";
    case FBQ_ERR_BADARG: return "bad argument";
    case FBQ_ERR_UNSUPPORTED: return "unsupported shape";
    case FBQ_ERR_ALIGN: return "pointer not 16-byte aligned";
    case FBQ_ERR_CUDA: return "CUDA runtime error";
    case FBQ_ERR_TIMEOUT: return "device-side wait expired";
    default: return "unknown status";
    }
}

}  // extern "C"
