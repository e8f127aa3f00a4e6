// Prefill kernel (M > 16) of the FBQuant linear, sm_100a: tcgen05 MMAs with the
// accumulator in tensor memory.
//
//   y = x.dequant(Q,s,z)^T + (x.A^T).B^T        (Algorithm 1 step 6 of the paper)
//
// At prefill the layer is a dense contraction, so it runs on the 5th-generation
// tensor cores.  One CTA owns a 128-token x 128-row output tile.  Four producer
// warps stream K in blocks of 64: each thread loads one token row of x and one
// packed weight row, dequantises the codes to the activation type (s*(q-z),
// q-z exact, one rounding) and writes both operands into shared memory in the
// K-major core-matrix layout the MMA reads (8 rows x 16 bytes per core matrix,
// no swizzle).  A fifth warp issues tcgen05.mma (128x128x16, fp32 accumulate in
// 128 TMEM columns) and hands stages back through tcgen05.commit.  The low-rank
// sub-branch is appended as extra K blocks of the same loop (Section 4.3 of the
// paper adds the up-projection into the shared output): their "x" operand is
// t = x.A^T, their "weight" operand is B as stored.  t itself comes from the
// same kernel run in down-projection mode (plain fp16/bf16 rows of A as the
// weight operand, K split over CTAs, fp32 atomics into scratch) one launch
// earlier; it is rounded once to the activation type when it is fed to the MMA.
// The producers' k order inside a block is permuted the same way for both
// operands (so that one LOP3 yields a finished pair of codes); a contraction
// does not care.  All waits are bounded.
#include "fbq_common.cuh"

namespace fbq {
namespace {

constexpr int kBM = 128, kBN = 128, kBK = 64;      // CTA tile (tokens, weight rows), K block
constexpr int kStages = 4;
constexpr int kProducers = 128;                    // threads 0..127: producers, then epilogue
constexpr int kPfThreads = kProducers + 32;        // + the MMA warp
constexpr uint32_t kStageBytes = 2u * kBM * kBK * 2u;          // x tile + weight tile, 16-bit elements
constexpr uint32_t kLBO = (kBM / 8) * 128;         // bytes between the two 8-element K chunks of an MMA
constexpr uint32_t kSBO = 128;                     // bytes between 8-row groups
constexpr uint32_t kPfWaitLimit = 1u << 20;
constexpr int kTmemCols = 128;

struct PrefillParams {
    const void *x;            // [M][K]
    const uint32_t *qw;       // packed codes (mode 0)
    const __half *scales;
    const __half *zeros;
    const void *Wplain;       // mode 1: A [rank][K];  mode 0: B [N][rank]
    float *t32;               // [M][rank] fp32: written (atomics) in mode 1, read in mode 0
    void *y;                  // [M][N] (mode 0)
    int *status;
    int M, N, K, rank;
    int kb_main;              // K / 64
    int kb_slab;              // ceil(rank / 64) (mode 0)
    int splitk;               // mode 1: number of K splits (grid.x)
};

// ---------------------------------------------------------------- PTX helpers
__device__ __forceinline__ uint32_t pf_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void pf_mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void pf_mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool pf_mbar_wait(uint32_t bar, uint32_t parity)
{
#pragma unroll 1
    for (uint32_t i = 0; i < kPfWaitLimit; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ void pf_fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory operand descriptor: K-major, no swizzle, core matrices of 8 rows x 16 bytes.
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr)
{
    return (uint64_t)((smem_addr >> 4) & 0x3FFFu) | ((uint64_t)(kLBO >> 4) << 16) | ((uint64_t)(kSBO >> 4) << 32) |
           (1ull << 46);
}
// D[tmem] (+)= A[smem] * B[smem]^T, 128 x 128 x 16, fp32 accumulate.
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive on an mbarrier once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t pf_lop3(uint32_t a, uint32_t mask, uint32_t orv)
{
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(a), "r"(mask), "r"(orv));   // (a & mask) | orv
    return r;
}
__device__ __forceinline__ uint32_t pf_prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}

// Packed-pair arithmetic of the activation type on raw 32-bit registers.
template <typename T> struct P2;
template <> struct P2<__half> {
    static constexpr uint32_t kFmt = 0;              // instruction-descriptor format code
    static __device__ __forceinline__ uint32_t sub(uint32_t a, uint32_t b)
    {
        uint32_t r;
        asm("sub.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
        return r;
    }
    static __device__ __forceinline__ uint32_t mul(uint32_t a, uint32_t b)
    {
        uint32_t r;
        asm("mul.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
        return r;
    }
    static __device__ __forceinline__ uint32_t fma(uint32_t a, uint32_t b, uint32_t c)
    {
        uint32_t r;
        asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
        return r;
    }
    static __device__ __forceinline__ uint32_t splat(float v)
    {
        __half2 h = __float2half2_rn(v);
        return *reinterpret_cast<uint32_t *>(&h);
    }
    static __device__ __forceinline__ uint32_t pack(float lo, float hi)
    {
        __half2 h = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<uint32_t *>(&h);
    }
};
template <> struct P2<__nv_bfloat16> {
    static constexpr uint32_t kFmt = 1;
    static __device__ __forceinline__ uint32_t sub(uint32_t a, uint32_t b)
    {
        uint32_t r;
        asm("sub.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
        return r;
    }
    static __device__ __forceinline__ uint32_t mul(uint32_t a, uint32_t b)
    {
        uint32_t r;
        asm("mul.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
        return r;
    }
    static __device__ __forceinline__ uint32_t fma(uint32_t a, uint32_t b, uint32_t c)
    {
        uint32_t r;
        asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
        return r;
    }
    static __device__ __forceinline__ uint32_t splat(float v)
    {
        __nv_bfloat162 h = __float2bfloat162_rn(v);
        return *reinterpret_cast<uint32_t *>(&h);
    }
    static __device__ __forceinline__ uint32_t pack(float lo, float hi)
    {
        __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t *>(&h);
    }
};

// Order of the 32 element pairs of one 64-wide K block as the dequantiser emits them
// (pair p occupies 32-bit word p of the block's shared-memory row).
template <int BITS> __device__ __forceinline__ constexpr int pair_lo(int p)
{
    if (BITS == 4) return 8 * (p / 4) + (p % 4);                       // word p/4: codes (e, e+4)
    const int r = p / 16, q = p % 16;                                  // run r of 32 codes
    return 32 * r + (q == 15 ? 30 : 10 * (q / 5) + (q % 5));
}
template <int BITS> __device__ __forceinline__ constexpr int pair_hi(int p)
{
    if (BITS == 4) return pair_lo<4>(p) + 4;
    const int r = p / 16, q = p % 16;
    return 32 * r + (q == 15 ? 31 : 10 * (q / 5) + 5 + (q % 5));
}

// s*(q - z) for the 64 codes of one weight row and K block, as 32 packed pairs in the
// order above.  q - z is exact (exponent trick, integer-valued z); the product is rounded
// once to the activation type.  w: 8 words (INT4) or 6 words (INT3).
template <int BITS, typename T> struct Dequant;
template <> struct Dequant<4, __half> {
    static __device__ __forceinline__ void run(const uint32_t *w, float s, float z, uint32_t *out)
    {
        const uint32_t c0 = P2<__half>::splat(1024.f + z), c1 = P2<__half>::splat(-(64.f + z)), s2 = P2<__half>::splat(s);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t a = w[i], b = w[i] >> 8;
            out[4 * i + 0] = P2<__half>::mul(P2<__half>::sub(pf_lop3(a, 0x000F000Fu, 0x64006400u), c0), s2);
            out[4 * i + 1] = P2<__half>::mul(P2<__half>::fma(pf_lop3(a, 0x00F000F0u, 0x64006400u), 0x2C002C00u, c1), s2);
            out[4 * i + 2] = P2<__half>::mul(P2<__half>::sub(pf_lop3(b, 0x000F000Fu, 0x64006400u), c0), s2);
            out[4 * i + 3] = P2<__half>::mul(P2<__half>::fma(pf_lop3(b, 0x00F000F0u, 0x64006400u), 0x2C002C00u, c1), s2);
        }
    }
};
template <> struct Dequant<4, __nv_bfloat16> {
    static __device__ __forceinline__ void run(const uint32_t *w, float s, float z, uint32_t *out)
    {
        using P = P2<__nv_bfloat16>;
        const uint32_t c0 = P::splat(128.f + z), s2 = P::splat(s);   // 0x4300 | q is 128 + q in bf16
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e)
                out[4 * i + e] = P::mul(P::sub(pf_lop3(w[i] >> (4 * e), 0x000F000Fu, 0x43004300u), c0), s2);
    }
};
template <> struct Dequant<3, __half> {
    static __device__ __forceinline__ void run(const uint32_t *w, float s, float z, uint32_t *out)
    {
        using P = P2<__half>;
        const uint32_t c0 = P::splat(1024.f + z), n1 = P::splat(-(128.f + z)), n2 = P::splat(-(16.f + z)), s2 = P::splat(s);
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const uint32_t *v = w + 3 * r;
            uint32_t *o = out + 16 * r;
#pragma unroll
            for (int i = 0; i < 3; ++i) {
                const uint32_t a = v[i], b = v[i] >> 9;
                o[5 * i + 0] = P::mul(P::sub(pf_lop3(a, 0x00070007u, 0x64006400u), c0), s2);
                o[5 * i + 1] = P::mul(P::fma(pf_lop3(a, 0x00380038u, 0x64006400u), 0x30003000u, n1), s2);
                o[5 * i + 2] = P::mul(P::fma(pf_lop3(a, 0x01C001C0u, 0x64006400u), 0x24002400u, n2), s2);
                o[5 * i + 3] = P::mul(P::sub(pf_lop3(b, 0x00070007u, 0x64006400u), c0), s2);
                o[5 * i + 4] = P::mul(P::fma(pf_lop3(b, 0x00380038u, 0x64006400u), 0x30003000u, n1), s2);
            }
            uint32_t l = pf_lop3(v[0] >> 15, 0x00010001u, 0x64006400u);
            l = pf_lop3(v[1] >> 14, 0x00020002u, l);
            l = pf_lop3(v[2] >> 13, 0x00040004u, l);
            o[15] = P::mul(P::sub(l, c0), s2);
        }
    }
};
template <> struct Dequant<3, __nv_bfloat16> {
    static __device__ __forceinline__ void run(const uint32_t *w, float s, float z, uint32_t *out)
    {
        using P = P2<__nv_bfloat16>;
        const uint32_t c0 = P::splat(128.f + z), n1 = P::splat(-(16.f + z)), s2 = P::splat(s);
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const uint32_t *v = w + 3 * r;
            uint32_t *o = out + 16 * r;
#pragma unroll
            for (int i = 0; i < 3; ++i) {
                const uint32_t a = v[i], b = v[i] >> 6, c = v[i] >> 12;
                o[5 * i + 0] = P::mul(P::sub(pf_lop3(a, 0x00070007u, 0x43004300u), c0), s2);
                o[5 * i + 1] = P::mul(P::fma(pf_lop3(a, 0x00380038u, 0x43004300u), 0x3E003E00u, n1), s2);
                o[5 * i + 2] = P::mul(P::sub(pf_lop3(b, 0x00070007u, 0x43004300u), c0), s2);
                o[5 * i + 3] = P::mul(P::fma(pf_lop3(b, 0x00380038u, 0x43004300u), 0x3E003E00u, n1), s2);
                o[5 * i + 4] = P::mul(P::sub(pf_lop3(c, 0x00070007u, 0x43004300u), c0), s2);
            }
            uint32_t l = pf_lop3(v[0] >> 15, 0x00010001u, 0x43004300u);
            l = pf_lop3(v[1] >> 14, 0x00020002u, l);
            l = pf_lop3(v[2] >> 13, 0x00040004u, l);
            o[15] = P::mul(P::sub(l, c0), s2);
        }
    }
};

// The same pair order applied to 64 natural-order 16-bit elements (8 x uint4).
template <int BITS> __device__ __forceinline__ void permute_pairs(const uint32_t *in /*32 words*/, uint32_t *out)
{
#pragma unroll
    for (int p = 0; p < 32; ++p) {
        const int lo = pair_lo<BITS>(p), hi = pair_hi<BITS>(p);
        const uint32_t sel = ((hi & 1) ? 0x7600u : 0x5400u) | ((lo & 1) ? 0x32u : 0x10u);
        out[p] = pf_prmt(in[lo >> 1], in[hi >> 1], sel);
    }
}

// One 64-element row of an operand tile goes to 8 core-matrix chunks of 16 bytes:
// chunk kc of row r lives at  kc*kLBO + (r/8)*kSBO + (r%8)*16.
__device__ __forceinline__ void store_row(uint8_t *tile, int r, const uint32_t *words /*32*/)
{
    uint8_t *base = tile + (r >> 3) * kSBO + (r & 7) * 16;
#pragma unroll
    for (int kc = 0; kc < 8; ++kc)
        *reinterpret_cast<uint4 *>(base + kc * kLBO) =
            make_uint4(words[4 * kc], words[4 * kc + 1], words[4 * kc + 2], words[4 * kc + 3]);
}

// --------------------------------------------------------------------- kernel
// MODE 0: y tile = x.dequant(W)^T + t.B^T  (grid: N tiles x M tiles)
// MODE 1: t32 += x.A^T over this CTA's K range (grid: K splits x M tiles), fp32 atomics
template <int MODE, int BITS, typename T>
__global__ void __launch_bounds__(kPfThreads, 1) prefill_kernel(const PrefillParams p)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t *stages = smem;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + (size_t)kStages * kStageBytes);
    const uint32_t full0 = pf_smem_u32(bars), empty0 = full0 + 8u * kStages, done_bar = empty0 + 8u * kStages;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * kStages + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.y * kBM;
    const int n0 = (MODE == 0) ? blockIdx.x * kBN : blockIdx.z * kBN;   // mode 1: tile of rank rows of A
    int kb_begin = 0, kb_end = p.kb_main + p.kb_slab;
    if (MODE == 1) {
        kb_begin = (int)((long long)blockIdx.x * p.kb_main / p.splitk);
        kb_end = (int)((long long)(blockIdx.x + 1) * p.kb_main / p.splitk);
    }
    const int nkb = kb_end - kb_begin;

    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) {
            pf_mbar_init(full0 + 8u * i, kProducers);
            pf_mbar_init(empty0 + 8u * i, 1);
        }
        pf_mbar_init(done_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kProducers / 32) {           // the MMA warp owns the tensor-memory allocation
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(pf_smem_u32(tmem_slot)),
                     "r"((uint32_t)kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        tc_fence_before();
    }
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp < kProducers / 32) {
        // =================================================== producers
        const int r = tid;                                  // row of both operand tiles
        const T *x = static_cast<const T *>(p.x);
        const int G = p.K / kGroupFast;
        bool dead = false;
#pragma unroll 1
        for (int i = 0; i < nkb && !dead; ++i) {
            const int kb = kb_begin + i, s = i % kStages;
            if (i >= kStages && !pf_mbar_wait(empty0 + 8u * s, (uint32_t)(i / kStages - 1) & 1u)) {
                dead = true;
                break;
            }
            if (*abort_flag) {
                dead = true;
                break;
            }
            uint32_t xa[32], wb[32];
            const int m = m0 + r;
            if (MODE == 1 || kb < p.kb_main) {
                uint32_t in[32];
                if (m < p.M) {
                    const uint4 *src = reinterpret_cast<const uint4 *>(x + (size_t)m * p.K + (size_t)kb * kBK);
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint4 v = __ldg(src + c);
                        in[4 * c] = v.x; in[4 * c + 1] = v.y; in[4 * c + 2] = v.z; in[4 * c + 3] = v.w;
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 32; ++c) in[c] = 0u;
                }
                if (MODE == 0) {
                    permute_pairs<BITS>(in, xa);
                    const int n = n0 + r;
                    if (n < p.N) {
                        constexpr int NW = (BITS == 4) ? 8 : 6;
                        uint32_t w[NW];
                        const uint32_t *src = p.qw + ((size_t)n * (p.K / kBK) + kb) * NW;
                        if (BITS == 4) {
                            const uint4 a = __ldg(reinterpret_cast<const uint4 *>(src)), b = __ldg(reinterpret_cast<const uint4 *>(src) + 1);
                            w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w; w[4] = b.x; w[5] = b.y; w[NW - 2] = b.z; w[NW - 1] = b.w;
                        } else {
#pragma unroll
                            for (int c = 0; c < 3; ++c) {
                                const uint2 a = __ldg(reinterpret_cast<const uint2 *>(src) + c);
                                w[2 * c] = a.x; w[2 * c + 1] = a.y;
                            }
                        }
                        const float sc = __half2float(p.scales[(size_t)n * G + kb / 2]);
                        const float ze = __half2float(p.zeros[(size_t)n * G + kb / 2]);
                        Dequant<BITS, T>::run(w, sc, ze, wb);
                    } else {
#pragma unroll
                        for (int c = 0; c < 32; ++c) wb[c] = 0u;
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 32; ++c) xa[c] = in[c];
                    if (n0 + r < p.rank) {                  // rows of A are the "weight" rows
                        const uint4 *src = reinterpret_cast<const uint4 *>(static_cast<const T *>(p.Wplain) + (size_t)(n0 + r) * p.K + (size_t)kb * kBK);
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            const uint4 v = __ldg(src + c);
                            wb[4 * c] = v.x; wb[4 * c + 1] = v.y; wb[4 * c + 2] = v.z; wb[4 * c + 3] = v.w;
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < 32; ++c) wb[c] = 0u;
                    }
                }
            } else {
                // sub-branch block: x operand = t (fp32 scratch, rounded once), weight operand = B as stored
                const int j0 = (kb - p.kb_main) * kBK;
                const int n = n0 + r;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const int j = j0 + 8 * c;
                    uint4 bv = make_uint4(0u, 0u, 0u, 0u);
                    float4 t0 = make_float4(0.f, 0.f, 0.f, 0.f), t1 = t0;
                    if (j < p.rank) {                       // rank is a multiple of 8: whole chunks
                        if (n < p.N) bv = __ldg(reinterpret_cast<const uint4 *>(static_cast<const T *>(p.Wplain) + (size_t)n * p.rank + j));
                        if (m < p.M) {
                            const float4 *ts = reinterpret_cast<const float4 *>(p.t32 + (size_t)m * p.rank + j);
                            t0 = __ldcg(ts);
                            t1 = __ldcg(ts + 1);
                        }
                    }
                    wb[4 * c] = bv.x; wb[4 * c + 1] = bv.y; wb[4 * c + 2] = bv.z; wb[4 * c + 3] = bv.w;
                    xa[4 * c] = P2<T>::pack(t0.x, t0.y); xa[4 * c + 1] = P2<T>::pack(t0.z, t0.w);
                    xa[4 * c + 2] = P2<T>::pack(t1.x, t1.y); xa[4 * c + 3] = P2<T>::pack(t1.z, t1.w);
                }
            }
            uint8_t *st = stages + (size_t)s * kStageBytes;
            store_row(st, r, xa);
            store_row(st + kBM * kBK * 2, r, wb);
            pf_fence_proxy_async();                         // generic-proxy stores -> visible to the MMA's reads
            pf_mbar_arrive(full0 + 8u * s);
        }
        if (dead) {
            *abort_flag = 1;
            atomicExch(p.status, (int)FBQ_ERR_TIMEOUT);
        }

        // =================================================== epilogue (same four warps)
        if (!dead && nkb > 0 && pf_mbar_wait(done_bar, 0)) {
            tc_fence_after();
            const int m = m0 + 32 * warp + lane;            // TMEM lane = token row of the tile
#pragma unroll 1
            for (int c = 0; c < kBN / 32; ++c) {
                uint32_t v[32];
                tc_ld32(tmem_base + ((uint32_t)(32 * warp) << 16) + (uint32_t)(32 * c), v);
                tc_wait_ld();
                if (m < p.M) {
                    if (MODE == 0) {
                        T *yrow = static_cast<T *>(p.y) + (size_t)m * p.N + n0 + 32 * c;
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            if (n0 + 32 * c + 8 * q < p.N) {     // N is a multiple of 8
                                uint4 o;
                                o.x = P2<T>::pack(__uint_as_float(v[8 * q + 0]), __uint_as_float(v[8 * q + 1]));
                                o.y = P2<T>::pack(__uint_as_float(v[8 * q + 2]), __uint_as_float(v[8 * q + 3]));
                                o.z = P2<T>::pack(__uint_as_float(v[8 * q + 4]), __uint_as_float(v[8 * q + 5]));
                                o.w = P2<T>::pack(__uint_as_float(v[8 * q + 6]), __uint_as_float(v[8 * q + 7]));
                                *reinterpret_cast<uint4 *>(yrow + 8 * q) = o;
                            }
                        }
                    } else {
#pragma unroll
                        for (int q = 0; q < 32; ++q) {
                            const int j = n0 + 32 * c + q;
                            if (j < p.rank) atomicAdd(p.t32 + (size_t)m * p.rank + j, __uint_as_float(v[q]));
                        }
                    }
                }
            }
        }
        tc_fence_before();
    } else {
        // =================================================== MMA warp
        constexpr uint32_t idesc = (1u << 4) | (P2<T>::kFmt << 7) | (P2<T>::kFmt << 10) | ((uint32_t)(kBN >> 3) << 17) |
                                   ((uint32_t)(kBM >> 4) << 24);
        bool dead = false;
#pragma unroll 1
        for (int i = 0; i < nkb && !dead; ++i) {
            const int s = i % kStages;
            if (lane == 0) {
                if (!pf_mbar_wait(full0 + 8u * s, (uint32_t)(i / kStages) & 1u) || *abort_flag) {
                    dead = true;
                } else {
                    tc_fence_after();
                    const uint32_t a_base = pf_smem_u32(stages + (size_t)s * kStageBytes), b_base = a_base + kBM * kBK * 2;
#pragma unroll
                    for (int j = 0; j < kBK / 16; ++j)
                        tc_mma(tmem_base, make_desc(a_base + j * 2 * kLBO), make_desc(b_base + j * 2 * kLBO), idesc,
                               (i > 0 || j > 0) ? 1u : 0u);
                    tc_commit(empty0 + 8u * s);              // stage is free once these MMAs have read it
                }
            }
            dead = __shfl_sync(0xffffffffu, (int)dead, 0) != 0;
        }
        if (lane == 0) {
            if (dead) {
                *abort_flag = 1;
                atomicExch(p.status, (int)FBQ_ERR_TIMEOUT);
            } else if (nkb > 0) {
                tc_commit(done_bar);                         // accumulator complete
            }
        }
        __syncwarp();
        tc_fence_before();
    }
    __syncthreads();
    if (warp == kProducers / 32) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
    }
}

constexpr size_t kPfSmem = (size_t)kStages * kStageBytes + (2 * kStages + 1) * 8 + 16;

template <int MODE, int BITS, typename T>
cudaError_t launch_mode(const PrefillParams &p, dim3 grid, cudaStream_t s)
{
    auto kern = prefill_kernel<MODE, BITS, T>;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPfSmem);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    kern<<<grid, kPfThreads, kPfSmem, s>>>(p);
    return cudaGetLastError();
}

template <typename T>
cudaError_t run_prefill(const LinearArgs &a, Workspace &ws, cudaStream_t s, int *launches)
{
    PrefillParams p{};
    p.x = a.x;
    p.qw = a.qw;
    p.scales = a.scales;
    p.zeros = a.zeros;
    p.t32 = ws.t_gen;
    p.y = a.y;
    p.status = ws.counters + kCtrStatus;
    p.M = a.M; p.N = a.N; p.K = a.K; p.rank = a.rank;
    p.kb_main = a.K / kBK;
    p.kb_slab = (a.rank + kBK - 1) / kBK;
    const unsigned mt = (unsigned)((a.M + kBM - 1) / kBM), nt = (unsigned)((a.N + kBN - 1) / kBN);
    cudaError_t e;
    if (a.rank > 0) {
        // t = x.A^T into fp32 scratch: K split so that about one CTA per SM is busy
        if ((e = cudaMemsetAsync(ws.t_gen, 0, sizeof(float) * (size_t)a.M * a.rank, s)) != cudaSuccess) return e;
        p.Wplain = a.A;
        p.splitk = (int)max(1u, min((unsigned)p.kb_main, 148u / mt));
        e = launch_mode<1, 4, T>(p, dim3((unsigned)p.splitk, mt, (unsigned)((a.rank + kBN - 1) / kBN)), s);
        if (e != cudaSuccess) return e;
        ++*launches;
    }
    p.Wplain = a.B;
    p.splitk = 1;
    e = (a.bits == 4) ? launch_mode<0, 4, T>(p, dim3(nt, mt), s) : launch_mode<0, 3, T>(p, dim3(nt, mt), s);
    if (e == cudaSuccess) ++*launches;
    return e;
}

}  // namespace

bool prefill_supported(const LinearArgs &a)
{
    return a.group == kGroupFast && a.K % kGroupFast == 0 && a.rank % 8 == 0 && a.rank <= kMaxRank && a.N % 8 == 0 &&
           a.M >= 1 && a.M <= 65535 * kBM;
}

// ws.t_gen must hold M x rank floats and ws.counters at least 8 ints (the caller grows them).
cudaError_t launch_prefill(const LinearArgs &a, Workspace &ws, cudaStream_t s, int *launches)
{
    if (!prefill_supported(a)) return cudaErrorInvalidConfiguration;
    return a.bf16 ? run_prefill<__nv_bfloat16>(a, ws, s, launches) : run_prefill<__half>(a, ws, s, launches);
}

}  // namespace fbq
