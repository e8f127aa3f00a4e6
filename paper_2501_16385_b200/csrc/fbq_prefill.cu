// Prefill kernel (M > 16) of the FBQuant linear, sm_100a: tcgen05 MMAs with the
// accumulator in tensor memory.
//
//   y = x.dequant(Q,s,z)^T + (x.A^T).B^T        (Algorithm 1 step 6 of the paper)
//
// At prefill the layer is a dense contraction, so it runs on the 5th-generation
// tensor cores.  One CTA owns a tile of 128 weight rows x TOK tokens (TOK = 256,
// or 128 for small M) and issues one 128 x TOK x 16 MMA per 16 elements of K:
// the weight tile is the MMA's A operand (its rows become the 128 TMEM lanes),
// the token tile the B operand (TOK fp32 columns).  Dequantising a weight tile
// once per 256 tokens halves the unpack work per flop against a 128-token tile,
// and the single wide MMA reads 96 bytes of shared memory per cycle, not 128.
//
// Every global read of the K loop is a TMA tensor copy (no multicast), so the
// load/store units only see shared memory:
//   * the token tile of a K block (64 elements of K) lands 128-byte swizzled,
//     ready for the MMA;
//   * the packed codes of the tile's 128 rows land, one quantisation group (two K
//     blocks) per copy, in a small ring that runs several groups ahead;
//   * in the sub-branch blocks the rows of B, and in down-projection mode the
//     rows of A, land 128-byte swizzled as the weight operand itself.
// Roles (20 warps):
//   warps 0-15  producers of the weight operand: warps 0-7 take the even groups,
//               warps 8-15 the odd ones; two threads per weight row, 32 codes of
//               each of the group's two K blocks per thread.  A thread reads its
//               words and (s, z) from the ring, dequantises to the activation type
//               (q - z exact by the exponent trick, one rounding in the product
//               with s), re-pairs the values into natural k order and stores them
//               as 128-byte rows in the same 128-byte swizzle the TMA copies use
//               (bank-conflict free for the stores and for the MMA's reads; the
//               no-swizzle core-matrix layout halved the MMA rate).  Afterwards the same warps drain the
//               accumulator: the tile is staged in shared memory and leaves with
//               TMA tensor stores (epilogue).
//   warp 16     one lane issues tcgen05.mma and hands stages back with
//               tcgen05.commit.
//   warp 17     one lane issues the operand-stage copies (token tile; B or A rows).
//   warps 18-19 keep the ring full: one lane issues the copies of packed codes;
//               all lanes read the tile's scales and zero points with 16-byte
//               loads (one per row and eight groups), realign them and write each
//               group's (s, z) words next to its ring slot.
// The low-rank sub-branch is appended as extra K blocks of the same loop
// (Section 4.3 of the paper adds the up-projection into the shared output):
// their token operand is t = x.A^T (fp32 scratch, rounded once to the activation
// type by the producers), their weight operand is B as stored.  t itself comes
// from the SAME launch: the first blocks of the grid run in down-projection mode
// (both operands by TMA, all of K or a K split each, plain fp32 stores to scratch)
// and raise a flag per token tile; the main CTAs look at the flag (bounded) only
// before their sub-branch blocks, at the very end of their K loop.
// All waits are bounded: a wait that runs out raises FBQ_ERR_TIMEOUT in the
// status word and every role falls through to the common exit.
#include <cuda.h>
#include <cudaTypedefs.h>

#include "fbq_common.cuh"

namespace fbq {
namespace {

constexpr int kBN = 128;                           // weight rows per CTA tile (MMA M)
constexpr int kBK = 64;                            // K block (one pipeline stage)
constexpr int kStages = 4;                         // operand stages
constexpr int kRing = 4;                           // groups of packed codes in flight
constexpr int kProducers = 512;                    // threads 0..511: producers, then epilogue
constexpr int kHalf = 256;                         // producers per group (two per weight row)
constexpr int kMmaWarp = kProducers / 32, kTmaWarp = kMmaWarp + 1, kRawWarp = kMmaWarp + 2;
constexpr int kPfThreads = kProducers + 128;         // + MMA warp, TMA warp, two ring warps
constexpr uint32_t kWBytes = kBN * kBK * 2u;       // weight operand tile of a stage
constexpr uint32_t kRawSlot = kBN * 64u;           // ring slot: 128 rows x one group of INT4 codes (INT3 uses 48 of 64)
constexpr int kPfCtrBase = 8;                      // first int of the workspace counters used for the t flags
constexpr uint32_t kPfWaitLimit = 1u << 20;
constexpr uint32_t kPfFlagPolls = 1u << 21;        // polls (256 ns apart) of a token tile's t flag: about half a second

struct PrefillParams {
    const __half *scales;     // [N][K/128]
    const __half *zeros;
    float *t32;               // [M][rank] fp32 scratch: written by the t CTAs, read by the main CTAs
    void *y;                  // [M][N]
    int *status;
    int M, N, K, rank;
    int kb_main;              // K / 64
    int kb_slab;              // ceil(rank / 64) (mode 0)
    int n_t;                  // number of t CTAs = token tiles x rank tiles (0 when rank == 0)
    int rt;                   // rank tiles of 128
    int nt;                   // feature tiles of 128
    int *tflag;               // [token tiles] warps of t CTAs that have stored their part (self-clearing)
    int *tdone;               // [token tiles] main CTAs that have consumed t (self-clearing)
    int splitk, splitt;       // K splits of a main tile / of a t tile (1 unless there are few tokens)
    float *part;              // [tile][split][128 rows][TOK] fp32 partial tiles (splitk > 1)
    int *split_ctr;           // [tile] splits that have stored their partial (self-clearing)
    uint32_t flag_polls;      // looks (256 ns apart) at a token tile's t flag before the wait gives up
    int test_skip_flag;       // test switch: the t CTAs do not raise the flag (the wait for t must run out)
    void *t16;                // [M][rank_pad] t rounded to the activation type, written by the t CTAs and read by the main
                              // CTAs' TMA copies as one more token operand (NULL: t32 and the producers' conversion)
    int rank_pad;             // columns of t16: rank rounded up to whole K blocks of 64 (the padding is zero)
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
__device__ __forceinline__ void pf_pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pf_fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory operand descriptor: K-major tile with 128-byte rows (64 16-bit elements) in the
// 128-byte swizzle (the 16-byte chunk c of row r is stored at chunk c ^ (r % 8)); groups of 8
// rows are 1024 bytes apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr)
{
    return (uint64_t)((smem_addr >> 4) & 0x3FFFu) | (1ull << 16) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// D[tmem] (+)= A[smem] * B[smem]^T, 128 x N x 16, fp32 accumulate.
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

// s*(q - z) for 32 consecutive codes of one weight row (half a K block), as 16 packed pairs
// in the order above.  q - z is exact (exponent trick, integer-valued z); the product is
// rounded once to the activation type.  w: 4 words (INT4) or one run of 3 words (INT3).
template <int BITS, typename T> struct Dequant;
template <> struct Dequant<4, __half> {
    static __device__ __forceinline__ void run(const uint32_t *w, float s, float z, uint32_t *out)
    {
        const uint32_t c0 = P2<__half>::splat(1024.f + z), c1 = P2<__half>::splat(-(64.f + z)), s2 = P2<__half>::splat(s);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
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
        for (int i = 0; i < 4; ++i)
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
        {
            const uint32_t *v = w;
            uint32_t *o = out;
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
        {
            const uint32_t *v = w;
            uint32_t *o = out;
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

// Where Dequant leaves element e (0..31, natural k order) of its 32 codes: register and half.
template <int BITS> __device__ __forceinline__ constexpr int elem_reg(int e)
{
    if (BITS == 4) return 4 * (e / 8) + (e % 4);                       // word e/8: pairs (j, j+4)
    const int r = e / 32, q = e % 32;                                  // run r of 32 codes
    return 16 * r + (q >= 30 ? 15 : 5 * (q / 10) + (q % 10) % 5);
}
template <int BITS> __device__ __forceinline__ constexpr int elem_half(int e)
{
    if (BITS == 4) return (e % 8) / 4;
    const int q = e % 32;
    return q >= 30 ? q - 30 : (q % 10) / 5;
}
// Re-pair the 32 dequantised values into natural order: word p = elements (2p, 2p+1).
template <int BITS> __device__ __forceinline__ void natural_pairs(const uint32_t *d /*16*/, uint32_t *out /*16*/)
{
#pragma unroll
    for (int p = 0; p < 16; ++p) {
        const int a = elem_reg<BITS>(2 * p), ha = elem_half<BITS>(2 * p);
        const int b = elem_reg<BITS>(2 * p + 1), hb = elem_half<BITS>(2 * p + 1);
        out[p] = pf_prmt(d[a], d[b], (hb ? 0x7600u : 0x5400u) | (ha ? 0x32u : 0x10u));
    }
}

template <typename T> __device__ __forceinline__ unsigned short to_bits16(float v)
{
    return (unsigned short)(P2<T>::pack(v, 0.f) & 0xFFFFu);
}

// --------------------------------------------------------------------- kernel
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void pf_mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// Shared-memory map of a CTA (byte offsets from the 1024-byte aligned base)
template <int TOK> struct Smem {
    static constexpr uint32_t kXBytes = (uint32_t)TOK * kBK * 2u;          // token operand tile of a stage
    static constexpr uint32_t kStageBytes = kXBytes + kWBytes;
    static constexpr uint32_t kRingOff = kStages * kStageBytes;
    static constexpr uint32_t kTableOff = kRingOff + kRing * kRawSlot;
    static constexpr uint32_t kBarOff = kTableOff + kRing * kBN * 4u;
    static constexpr uint32_t kNumBars = 2 * kStages + 2 * kRing + 1 + 4 + 2;  // full, empty, ring full, ring empty, done, epilogue, split
    static constexpr uint32_t kTotal = kBarOff + kNumBars * 8u + 16u;
};

// One launch, 1-D grid.  The first n_t CTAs are "t CTAs": CTA (token tile, rank tile) computes
// t = x.A^T for 256 tokens x 128 rank indices over all of K (both operands by TMA) and stores it as
// fp32 to scratch, then raises the token tile's flag.  The other CTAs are main CTAs, one per
// (feature tile, token tile): y tile = x.dequant(W)^T + t.B^T; they look at the flag only before
// their sub-branch blocks, at the very end of the K loop, by which time the t CTAs (lowest block
// indices, so dispatched first, and with no unpacking to do) have long finished.  The wait is
// bounded like all others.  The last main CTA of a token tile to finish clears the flag again.
// xmap: x [M][K], boxes of TOK rows x 64 elements, 128-byte swizzle
// wmap: packed codes [N][words per row], boxes of 128 rows x one group (64-byte swizzle for INT4)
// amap: A [rank][K], boxes of 128 rows x 64 elements, 128-byte swizzle (t CTAs)
// bmap: B [N][rank], boxes of 128 rows x 64 elements, 128-byte swizzle (main CTAs, rank > 0)
// ymap: y [M][N], boxes of TOK/4 rows x 128 elements, no swizzle (stores)
// tmap: t16 [M][rank_pad], boxes like xmap's (main CTAs, rank > 0, one K split of t)
template <int BITS, typename T, int TOK>
__global__ void __launch_bounds__(kPfThreads, 1)
prefill_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap wmap,
               const __grid_constant__ CUtensorMap amap, const __grid_constant__ CUtensorMap bmap,
               const __grid_constant__ CUtensorMap ymap, const __grid_constant__ CUtensorMap tmap, const PrefillParams p)
{
    using L = Smem<TOK>;
    constexpr uint32_t kXBytes = L::kXBytes, kStageBytes = L::kStageBytes;
    constexpr int WPG = (BITS == 4) ? 16 : 12;                  // packed words per row and group
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = pf_smem_u32(smem);
    if (sbase & 1023u) {                                        // swizzle atoms need a 1024-byte aligned base
        if (threadIdx.x == 0) atomicExch(p.status, (int)FBQ_ERR_CUDA);
        return;
    }
    const uint32_t full0 = sbase + L::kBarOff, empty0 = full0 + 8u * kStages, rfull0 = empty0 + 8u * kStages,
                   rempty0 = rfull0 + 8u * kRing, done_bar = rempty0 + 8u * kRing, epi0 = done_bar + 8u,
                   split_bar = epi0 + 32u, split_bar2 = split_bar + 8u;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + L::kBarOff + L::kNumBars * 8u);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    volatile int *split_last = abort_flag + 1;                  // 1: this CTA adds up the K splits of its tile

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool t_role = (int)blockIdx.x < p.n_t;                // t CTA or main CTA
    // (token tile, feature or rank tile, K split): with few tokens there are few tiles, so K is split over
    // several CTAs per tile (splitk main CTAs whose fp32 partial tiles the last one to finish adds up,
    // splitt t CTAs that each store their own partial t)
    int m_tile, n_tile, split;
    const int S = t_role ? p.splitt : p.splitk;
    {
        int b = t_role ? (int)blockIdx.x : (int)blockIdx.x - p.n_t;
        split = b % S;
        b /= S;
        const int tiles = t_role ? p.rt : p.nt;
        m_tile = b / tiles;
        n_tile = b % tiles;
    }
    const int m0 = m_tile * TOK, n0 = n_tile * kBN;
    const int G_all = p.kb_main >> 1;
    const int g_begin = (int)((long long)split * G_all / S), g_end = (int)((long long)(split + 1) * G_all / S);
    const int kb_begin = 2 * g_begin;                           // first K block of this CTA's range
    const int kb_x = 2 * (g_end - g_begin);                     // blocks [0, kb_x) of the CTA take their tokens from x
    const int nkb = kb_x + ((t_role || split != 0) ? 0 : p.kb_slab);     // the sub-branch blocks go to split 0

    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) {
            pf_mbar_init(full0 + 8u * i, t_role ? 1 : kHalf / 32 + 1);   // 8 producer warps + the TMA lane
            pf_mbar_init(empty0 + 8u * i, 1);
        }
        for (int i = 0; i < kRing; ++i) {
            pf_mbar_init(rfull0 + 8u * i, 2);                   // the two ring warps
            pf_mbar_init(rempty0 + 8u * i, kHalf / 32);         // a group is consumed by one half of the producers (8 warps)
        }
        pf_mbar_init(done_bar, 1);
        for (int i = 0; i < 4; ++i) pf_mbar_init(epi0 + 8u * i, 128);     // the four warps of a column quarter
        pf_mbar_init(split_bar, kProducers / 32);               // every epilogue warp has stored its partial chunk
        pf_mbar_init(split_bar2, 1);                            // warp 0 has counted the CTA in
        *abort_flag = 0;
        *split_last = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kMmaWarp) {                  // the MMA warp owns the tensor-memory allocation
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(pf_smem_u32(tmem_slot)),
                     "r"((uint32_t)TOK)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        tc_fence_before();
    }
    if (warp == kTmaWarp && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&xmap)) : "memory");
        if (t_role) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&amap)) : "memory");
        } else {
            if (p.rank > 0) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&bmap)) : "memory");
            if (p.t16) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap)) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&ymap)) : "memory");
        }
    }
    if (warp == kRawWarp && lane == 0)
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&wmap)) : "memory");
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // Programmatic dependent launch: the CTAs of the launch that follows may take their SMs as soon as ours leave
    // them and run their own set-up above; nothing before this point reads or writes global memory, everything
    // after it waits for the preceding launch to have completed (so no bounded wait below spans that launch).
    // Letting the ring of packed codes and the first two dequantised groups start before the wait was measured
    // and changed nothing (68.8 against 68.9 us per linear of a layer step).
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    pf_pdl_wait();

    if (warp < kMmaWarp) {
        bool dead = false;
        if (!t_role) {
            // =================================================== producers
            // Half h of the warps takes the groups g = h, h+2, ... (K blocks 2g and 2g+1, stages 2h
            // and 2h+1); thread (row r, part) dequantises the codes [32*part, +32) of both blocks.
            const int h = warp >> 3, part = (warp >> 2) & 1, r = tid & 127;
            const bool row_ok = n0 + r < p.N;
            const int groups = kb_x >> 1;
            // this thread's words inside a ring slot: block b holds codes [64b, 64b+64) of the group
            uint32_t roff0, roff1;
            if (BITS == 4) {                                // 64-byte rows, 16-byte chunk c stored at c ^ ((row / 2) % 4)
                const uint32_t sw = (uint32_t)(r >> 1) & 3u;
                roff0 = (uint32_t)r * 64u + ((((uint32_t)part) ^ sw) << 4);
                roff1 = (uint32_t)r * 64u + ((((uint32_t)part + 2u) ^ sw) << 4);
            } else {                                        // 48-byte rows of four 12-byte runs
                roff0 = (uint32_t)r * 48u + (uint32_t)part * 12u;
                roff1 = roff0 + 24u;
            }
            const uint32_t ring0 = sbase + L::kRingOff, table0 = sbase + L::kTableOff + (uint32_t)r * 4u;
            // weight tile rows are 128 bytes (64 elements); the 16-byte chunk c of row r sits at c ^ (r % 8)
            const uint32_t wdst = sbase + kXBytes + (uint32_t)(2 * h) * kStageBytes + (uint32_t)r * 128u;
            const uint32_t wsw = (uint32_t)r & 7u;
            const uint32_t fullb = full0 + 16u * h, emptyb = empty0 + 16u * h;
            uint32_t slot = (uint32_t)h, rphase = 0u, ephase = 0u;
#pragma unroll 1
            for (int g = h; g < groups; g += 2) {
                if (!pf_mbar_wait(rfull0 + 8u * slot, rphase)) { dead = true; break; }
                constexpr int NW = (BITS == 4) ? 4 : 3;
                uint32_t w[2][NW];
                const uint32_t rs = ring0 + slot * kRawSlot;
                if (BITS == 4) {
                    const uint4 a = lds128(rs + roff0), b = lds128(rs + roff1);
                    w[0][0] = a.x; w[0][1] = a.y; w[0][2] = a.z; w[0][NW - 1] = a.w;
                    w[1][0] = b.x; w[1][1] = b.y; w[1][2] = b.z; w[1][NW - 1] = b.w;
                } else {
#pragma unroll
                    for (int c = 0; c < 3; ++c) {
                        w[0][c] = lds32(rs + roff0 + 4u * c);
                        w[1][c] = lds32(rs + roff1 + 4u * c);
                    }
                }
                const uint32_t sz = lds32(table0 + slot * (kBN * 4u));      // s | z << 16 of (row, group)
                __syncwarp();
                if (lane == 0) pf_mbar_arrive(rempty0 + 8u * slot);   // the warp's words are in registers: the slot may be refilled
                slot += 2u;
                if (slot >= (uint32_t)kRing) { slot -= (uint32_t)kRing; rphase ^= 1u; }
                const float sc = __half2float(__ushort_as_half((unsigned short)(sz & 0xFFFFu)));
                const float ze = __half2float(__ushort_as_half((unsigned short)(sz >> 16)));
#pragma unroll
                for (int b = 0; b < 2; ++b) {
                    if (g >= 2 && !pf_mbar_wait(emptyb + 8u * b, ephase)) { dead = true; break; }
                    uint32_t wb[16];
                    if (row_ok) {
                        uint32_t d[16];
                        Dequant<BITS, T>::run(w[b], sc, ze, d);
                        natural_pairs<BITS>(d, wb);
                    } else {
#pragma unroll
                        for (int c = 0; c < 16; ++c) wb[c] = 0u;
                    }
#pragma unroll
                    for (int kc = 0; kc < 4; ++kc)
                        sts128(wdst + (uint32_t)b * kStageBytes + ((((uint32_t)(4 * part + kc)) ^ wsw) << 4), wb[4 * kc], wb[4 * kc + 1], wb[4 * kc + 2],
                               wb[4 * kc + 3]);
                }
                if (dead) break;
                pf_fence_proxy_async();                     // generic-proxy stores -> visible to the MMA's reads
                __syncwarp();
                if (lane == 0) {                            // one arrival per warp and block
                    pf_mbar_arrive(fullb);
                    pf_mbar_arrive(fullb + 8u);
                }
                if (g >= 2) ephase ^= 1u;
            }
            // ---- sub-branch blocks: token operand = t (fp32 scratch, rounded once); B arrives by TMA.
            // The halves take them in turn, one token row per thread.
            bool t_ready = false;
#pragma unroll 1
            for (int i = kb_x + h; i < nkb && !dead; i += 2) {
                const int s = i % kStages;
                if (i >= kStages && !pf_mbar_wait(empty0 + 8u * s, (uint32_t)(i / kStages - 1) & 1u)) { dead = true; break; }
                if (p.t16) {                                 // both operands of this block arrive by TMA: nothing to write
                    __syncwarp();
                    if (lane == 0) pf_mbar_arrive(full0 + 8u * s);
                    continue;
                }
                if (!t_ready) {                              // every warp of every t CTA of this token tile has stored its part
                    int seen = 0;
                    if (lane == 0) {
                        const int *flag = p.tflag + m_tile;
                        const int target = 16 * p.rt * p.splitt;
#pragma unroll 1
                        for (uint32_t spin = 0; spin < p.flag_polls; ++spin) {
                            asm volatile("ld.acquire.gpu.global.b32 %0, [%1];" : "=r"(seen) : "l"(flag) : "memory");
                            if (seen >= target) break;
                            __nanosleep(256);
                        }
                        seen = seen >= target;
                    }
                    t_ready = __shfl_sync(0xffffffffu, seen, 0) != 0;
                    if (!t_ready) { dead = true; break; }
                }
                const int j0 = (i - kb_x) * kBK;
                const int rr = tid & (kHalf - 1);            // token row of the tile
                if (rr < TOK) {
                    const int m = m0 + rr;
                    uint32_t xa[32];
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        float4 t0 = make_float4(0.f, 0.f, 0.f, 0.f), t1 = t0;
                        if (m < p.M && j0 + 8 * c < p.rank) {              // rank is a multiple of 8: whole chunks
                            const float4 *ts = reinterpret_cast<const float4 *>(p.t32 + (size_t)m * p.rank + j0 + 8 * c);
                            t0 = __ldcg(ts);
                            t1 = __ldcg(ts + 1);
                            for (int sp = 1; sp < p.splitt; ++sp) {         // partial t of the other K splits, in order
                                const float4 *us = ts + (size_t)sp * p.M * p.rank / 4;
                                const float4 u0 = __ldcg(us), u1 = __ldcg(us + 1);
                                t0.x += u0.x; t0.y += u0.y; t0.z += u0.z; t0.w += u0.w;
                                t1.x += u1.x; t1.y += u1.y; t1.z += u1.z; t1.w += u1.w;
                            }
                        }
                        xa[4 * c] = P2<T>::pack(t0.x, t0.y); xa[4 * c + 1] = P2<T>::pack(t0.z, t0.w);
                        xa[4 * c + 2] = P2<T>::pack(t1.x, t1.y); xa[4 * c + 3] = P2<T>::pack(t1.z, t1.w);
                    }
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        sts128(sbase + (uint32_t)s * kStageBytes + (uint32_t)rr * 128u + ((((uint32_t)c) ^ ((uint32_t)rr & 7u)) << 4), xa[4 * c],
                               xa[4 * c + 1], xa[4 * c + 2], xa[4 * c + 3]);
                }
                pf_fence_proxy_async();
                __syncwarp();
                if (lane == 0) pf_mbar_arrive(full0 + 8u * s);
            }
            if (dead) {
                *abort_flag = 1;
                atomicExch(p.status, (int)FBQ_ERR_TIMEOUT);
            }
        }

        // =================================================== epilogue (same sixteen warps)
        // TMEM lane = weight row of the tile, column = token.  Warp w reads lanes 32*(w%4)..+31
        // (the only ones it may address) and the quarter w/4 of the columns.  Mode 0 stages the
        // tile in shared memory as [token][128 features] (the operand stages are free by now) and
        // each column quarter leaves with one TMA tensor store, which also clips the ragged edges.
        if (!dead && nkb > 0 && pf_mbar_wait(done_bar, 0)) {
            tc_fence_after();
            const int q = warp & 3, cg = warp >> 2;
            const int nn = n0 + 32 * q + lane;              // output feature (mode 0) / rank index (mode 1)
            const int c_begin = cg * (TOK / 4);
            if (!t_role && S > 1) {
                // ---- K split over S CTAs (TOK = 128: one 32-column chunk per warp).  Every CTA stores its
                // fp32 partial tile; the CTA that counts in last adds the S partials in split order (the
                // result does not depend on which CTA that is) and is the one that writes y.
                const bool mine = m0 + c_begin < p.M;       // uniform over the four warps of a column quarter
                const size_t slice = (size_t)kBN * TOK;
                float *pt = p.part + ((size_t)(m_tile * p.nt + n_tile) * S) * slice + (size_t)(32 * q + lane) * TOK + c_begin;
                uint32_t v[32];
                if (mine) {
                    tc_ld32(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)c_begin, v);
                    tc_wait_ld();
                    float4 *dst = reinterpret_cast<float4 *>(pt + (size_t)split * slice);
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        __stcg(dst + j, make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                                    __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3])));
                }
                __threadfence();
                __syncwarp();
                if (lane == 0) pf_mbar_arrive(split_bar);
                if (warp == 0 && lane == 0) {
                    int last = 0;
                    if (pf_mbar_wait(split_bar, 0)) {
                        int *ctr = p.split_ctr + m_tile * p.nt + n_tile;
                        last = (atomicAdd(ctr, 1) == S - 1);
                        if (last) atomicExch(ctr, 0);       // left at zero for the next call
                    } else {
                        atomicExch(p.status, (int)FBQ_ERR_TIMEOUT);
                    }
                    *split_last = last;
                    __threadfence_block();
                    pf_mbar_arrive(split_bar2);
                }
                const bool last = pf_mbar_wait(split_bar2, 0) && *split_last != 0;
                if (last && mine) {
                    __threadfence();
                    float acc[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) acc[j] = 0.f;
#pragma unroll 1
                    for (int sp = 0; sp < S; ++sp) {
                        const float4 *src = reinterpret_cast<const float4 *>(pt + (size_t)sp * slice);
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const float4 u = __ldcg(src + j);
                            acc[4 * j] += u.x; acc[4 * j + 1] += u.y; acc[4 * j + 2] += u.z; acc[4 * j + 3] += u.w;
                        }
                    }
                    unsigned short *sp16 = reinterpret_cast<unsigned short *>(smem + (size_t)c_begin * (kBN * 2)) + 32 * q + lane;
#pragma unroll
                    for (int j = 0; j < 32; ++j) sp16[j * kBN] = to_bits16<T>(acc[j]);
                    pf_fence_proxy_async();                 // staged tile -> visible to the TMA store
                    pf_mbar_arrive(epi0 + 8u * cg);
                    if (q == 0 && lane == 0) {
                        if (pf_mbar_wait(epi0 + 8u * cg, 0)) {
                            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                                         ::"l"(reinterpret_cast<uint64_t>(&ymap)), "r"(n0), "r"(m0 + c_begin),
                                           "r"(sbase + (uint32_t)c_begin * (kBN * 2))
                                         : "memory");
                            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                        } else {
                            atomicExch(p.status, (int)FBQ_ERR_TIMEOUT);
                        }
                    }
                }
            } else if (m0 + c_begin < p.M) {                // uniform over the four warps of a column quarter
#pragma unroll 1
                for (int c = c_begin; c < c_begin + TOK / 4; c += 32) {
                    if (m0 + c >= p.M) break;               // warp-uniform
                    uint32_t v[32];
                    tc_ld32(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)c, v);
                    tc_wait_ld();
                    if (!t_role) {
                        unsigned short *sp = reinterpret_cast<unsigned short *>(smem + (size_t)c * (kBN * 2)) + 32 * q + lane;
#pragma unroll
                        for (int j = 0; j < 32; ++j) sp[j * kBN] = to_bits16<T>(__uint_as_float(v[j]));
                    } else if (p.t16) {
                        if (nn < p.rank_pad) {               // rounded once, here; rows of A beyond the rank are zero fill
                            unsigned short *tp = static_cast<unsigned short *>(p.t16) + (size_t)(m0 + c) * p.rank_pad + nn;
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (m0 + c + j < p.M) tp[(size_t)j * p.rank_pad] = to_bits16<T>(__uint_as_float(v[j]));
                        }
                    } else {
                        if (nn < p.rank) {                   // 32 lanes = 32 consecutive rank indices: 128-byte stores
                            float *tp = p.t32 + (size_t)split * p.M * p.rank + (size_t)(m0 + c) * p.rank + nn;
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (m0 + c + j < p.M) __stcg(tp + (size_t)j * p.rank, __uint_as_float(v[j]));
                        }
                    }
                }
                if (!t_role) {
                    pf_fence_proxy_async();                 // staged tile -> visible to the TMA store
                    pf_mbar_arrive(epi0 + 8u * cg);
                    if (q == 0 && lane == 0) {
                        if (pf_mbar_wait(epi0 + 8u * cg, 0)) {
                            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                                         ::"l"(reinterpret_cast<uint64_t>(&ymap)), "r"(n0), "r"(m0 + c_begin),
                                           "r"(sbase + (uint32_t)c_begin * (kBN * 2))
                                         : "memory");
                            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // smem may go once it has been read
                        } else {
                            atomicExch(p.status, (int)FBQ_ERR_TIMEOUT);
                        }
                    }
                }
            }
            if (t_role) {
                // this warp's part of t is stored: make it visible (to the main CTAs' TMA copies as well), then count the warp in
                asm volatile("fence.proxy.async;" ::: "memory");
                __threadfence();
                __syncwarp();
                if (lane == 0 && !p.test_skip_flag) atomicAdd(p.tflag + m_tile, 1);
            } else if (p.rank > 0 && tid == 0 && split == 0) {
                // this CTA has consumed t (its MMAs are complete).  The last main CTA of the token
                // tile leaves the flag and the count at zero for the next call.
                if (atomicAdd(p.tdone + m_tile, 1) == p.nt - 1) {
                    atomicExch(p.tflag + m_tile, 0);
                    atomicExch(p.tdone + m_tile, 0);
                }
            }
        }
        tc_fence_before();
    } else if (warp == kMmaWarp) {
        // =================================================== MMA warp
        constexpr uint32_t idesc = (1u << 4) | (P2<T>::kFmt << 7) | (P2<T>::kFmt << 10) | ((uint32_t)(TOK >> 3) << 17) |
                                   ((uint32_t)(kBN >> 4) << 24);
        bool dead = false;
#pragma unroll 1
        for (int i = 0; i < nkb && !dead; ++i) {
            const int s = i % kStages;
            if (lane == 0) {
                if (!pf_mbar_wait(full0 + 8u * s, (uint32_t)(i / kStages) & 1u) || *abort_flag) {
                    dead = true;
                } else {
                    tc_fence_after();
                    const uint32_t x_base = sbase + (uint32_t)s * kStageBytes, w_base = x_base + kXBytes;
                    // every operand tile is K-major with 128-byte rows and the 128-byte swizzle, whether it
                    // arrived by TMA or was written by the producers: 32 bytes per 16 elements of K inside a row
#pragma unroll
                    for (int j = 0; j < kBK / 16; ++j)
                        tc_mma(tmem_base, make_desc(w_base + j * 32), make_desc(x_base + j * 32), idesc, (i > 0 || j > 0) ? 1u : 0u);
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
    } else if (warp == kTmaWarp) {
        // =================================================== operand-stage copies
        if (lane == 0) {
            bool dead = false;
#pragma unroll 1
            for (int i = 0; i < nkb; ++i) {
                const int kb = i, s = i % kStages;
                if ((i >= kStages && !pf_mbar_wait(empty0 + 8u * s, (uint32_t)(i / kStages - 1) & 1u)) || *abort_flag) {
                    dead = true;
                    break;
                }
                const uint32_t bar = full0 + 8u * s;
                const uint32_t xt = sbase + (uint32_t)s * kStageBytes, wt = xt + kXBytes;
                if (t_role) {
                    pf_mbar_expect_tx(bar, kXBytes + kWBytes);
                    tma_load_2d(xt, &xmap, (kb_begin + kb) * kBK, m0, bar);
                    tma_load_2d(wt, &amap, (kb_begin + kb) * kBK, n0, bar);      // rows of A
                } else if (kb < kb_x) {
                    pf_mbar_expect_tx(bar, kXBytes);
                    tma_load_2d(xt, &xmap, (kb_begin + kb) * kBK, m0, bar);
                } else if (p.t16) {
                    if (kb == kb_x) {                        // every warp of every t CTA of this token tile has stored its part
                        const int *flag = p.tflag + m_tile;
                        const int target = 16 * p.rt * p.splitt;
                        int seen = 0;
#pragma unroll 1
                        for (uint32_t spin = 0; spin < p.flag_polls; ++spin) {
                            asm volatile("ld.acquire.gpu.global.b32 %0, [%1];" : "=r"(seen) : "l"(flag) : "memory");
                            if (seen >= target) break;
                            __nanosleep(256);
                        }
                        if (seen < target) {
                            dead = true;
                            break;
                        }
                        asm volatile("fence.proxy.async;" ::: "memory");
                    }
                    pf_mbar_expect_tx(bar, kXBytes + kWBytes);
                    tma_load_2d(xt, &tmap, (kb - kb_x) * kBK, m0, bar);   // t as the token operand
                    tma_load_2d(wt, &bmap, (kb - kb_x) * kBK, n0, bar);   // rows of B
                } else {
                    pf_mbar_expect_tx(bar, kWBytes);
                    tma_load_2d(wt, &bmap, (kb - kb_x) * kBK, n0, bar);   // rows of B
                }
            }
            if (dead) {
                *abort_flag = 1;
                atomicExch(p.status, (int)FBQ_ERR_TIMEOUT);
                for (int i = 0; i < 64; ++i) __nanosleep(1000);   // let the copies in flight land before the CTA exits
            }
        }
        __syncwarp();
    } else if (!t_role) {
        // =================================================== ring of packed codes and (s, z) table
        // Two warps; lane l of ring warp v owns the tile rows 64v + l and 64v + l + 32.  Per chunk of
        // eight groups it reads the rows' scales and zero points with 16-byte loads (two aligned chunks of the flat row-major arrays
        // cover any eight consecutive values), realigns them in registers, and before each group's
        // copy writes that group's (s | z << 16) words next to the ring slot.
        const int G = p.K / kGroupFast, groups = kb_x >> 1;     // all groups of a row; groups of this CTA's K range
        const size_t n_chunks = (size_t)p.N * G / 8;        // N is a multiple of 8
        const uint4 *s_arr = reinterpret_cast<const uint4 *>(p.scales), *z_arr = reinterpret_cast<const uint4 *>(p.zeros);
        const int v = warp - kRawWarp;
        size_t a0[2];                                       // aligned 16-byte chunk holding group 0 of the row
        uint32_t off[2];                                    // position of group 0 inside that chunk (0..7)
        bool ok[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const int n = n0 + 64 * v + lane + 32 * k;
            ok[k] = n < p.N;
            const size_t f = (size_t)(ok[k] ? n : 0) * G + g_begin;      // first group of this CTA's range
            a0[k] = f >> 3;
            off[k] = (uint32_t)f & 7u;
        }
        uint4 raw[2][2][2];                                 // [row][s|z][low|high chunk] of the next eight groups
        auto fetch = [&](int c) {
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const size_t a = a0[k] + (size_t)c;
                const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
                raw[k][0][0] = (ok[k] && a < n_chunks) ? __ldg(s_arr + a) : zero;
                raw[k][1][0] = (ok[k] && a < n_chunks) ? __ldg(z_arr + a) : zero;
                raw[k][0][1] = (ok[k] && a + 1 < n_chunks) ? __ldg(s_arr + a + 1) : zero;
                raw[k][1][1] = (ok[k] && a + 1 < n_chunks) ? __ldg(z_arr + a + 1) : zero;
            }
        };
        // eight consecutive fp16 values starting `o` values into the 16-value window (lo, hi), as 4 pair-words
        auto realign = [](const uint4 &lo, const uint4 &hi, uint32_t o, uint32_t (&out)[4]) {
            uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
            if (o & 2u) {
#pragma unroll
                for (int i = 0; i < 7; ++i) w[i] = w[i + 1];
            }
            if (o & 4u) {
#pragma unroll
                for (int i = 0; i < 5; ++i) w[i] = w[i + 2];
            }
#pragma unroll
            for (int t = 0; t < 4; ++t) out[t] = __funnelshift_r(w[t], w[t + 1], (o & 1u) * 16u);
        };
        bool dead = false;
        const uint32_t ring0 = sbase + L::kRingOff, table0 = sbase + L::kTableOff + (uint32_t)(64 * v + lane) * 4u;
        fetch(0);
#pragma unroll 1
        for (int c = 0; 8 * c < groups && !dead; ++c) {
            uint32_t sz[2][8];                              // (s | z << 16) of [row][group of this chunk]
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                uint32_t sp[4], zp[4];
                realign(raw[k][0][0], raw[k][0][1], off[k], sp);
                realign(raw[k][1][0], raw[k][1][1], off[k], zp);
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    sz[k][2 * t] = pf_prmt(sp[t], zp[t], 0x5410u);
                    sz[k][2 * t + 1] = pf_prmt(sp[t], zp[t], 0x7632u);
                }
            }
            if (8 * (c + 1) < groups) fetch(c + 1);
#pragma unroll
            for (int g8 = 0; g8 < 8; ++g8) {
                const int gi = 8 * c + g8;
                if (gi < groups && !dead) {
                    const uint32_t slot = (uint32_t)gi % kRing;
                    if (lane == 0 && ((gi >= kRing && !pf_mbar_wait(rempty0 + 8u * slot, (uint32_t)(gi / kRing - 1) & 1u)) || *abort_flag))
                        dead = true;
                    dead = __shfl_sync(0xffffffffu, (int)dead, 0) != 0;     // also orders the table writes after the wait
                    if (!dead) {
#pragma unroll
                        for (int k = 0; k < 2; ++k)
                            asm volatile("st.shared.b32 [%0], %1;" ::"r"(table0 + slot * (kBN * 4u) + 128u * k), "r"(sz[k][g8]) : "memory");
                        __syncwarp();
                        if (lane == 0) {
                            if (v == 0) {
                                pf_mbar_expect_tx(rfull0 + 8u * slot, (uint32_t)kBN * WPG * 4u);
                                tma_load_2d(ring0 + slot * kRawSlot, &wmap, (g_begin + gi) * WPG, n0, rfull0 + 8u * slot);
                            } else {
                                pf_mbar_arrive(rfull0 + 8u * slot);
                            }
                        }
                    }
                }
            }
        }
        if (dead && lane == 0) {
            *abort_flag = 1;
            atomicExch(p.status, (int)FBQ_ERR_TIMEOUT);
            for (int i = 0; i < 64; ++i) __nanosleep(1000);
        }
        __syncwarp();
    }
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TOK) : "memory");
    }
}

// ---------------------------------------------------------------- CTA-pair variant
// Two CTAs of a cluster (two SMs) share one MMA of 256 weight rows x 256 tokens x 16
// (tcgen05 cta_group::2): each CTA dequantises its own 128 weight rows and stages only HALF of
// the token tile (128 tokens); the tensor cores of both SMs read both halves.  Per CTA and K
// block that is 16 KB less written by TMA and 16 KB less read by the MMA than in the single-CTA
// kernel, and it leaves room for six stages.  MEASURED SLOWER than the single-CTA kernel on B200
// (M = 1024, 4096 -> 4096, INT4, bf16: 47.8 us against 39.8 us; 1120 against 880 cycles per K
// block; with dequantisation, copies and MMAs all switched off the bare hand-shake still takes 760
// cycles per block: the round trip peer arrival -> leader -> multicast commit -> peer is about
// 4500 cycles, more than six stages of MMA time cover), so it is off by default ("prefill_pair"
// option) and kept as a checked alternative.
// The leader CTA (cluster rank 0) issues every MMA; all arrivals that say "stage full" (the
// producer warps of both CTAs, the byte counts of both CTAs' TMA copies) go to the leader's
// barriers; tcgen05.commit with a cluster multicast frees the stage in both CTAs.
constexpr int kPairStages = 6;
struct PairSmem {
    static constexpr uint32_t kXBytes = 128u * kBK * 2u;                   // this CTA's half of the token tile
    static constexpr uint32_t kStageBytes = kXBytes + kWBytes;
    static constexpr uint32_t kRingOff = kPairStages * kStageBytes;
    static constexpr uint32_t kTableOff = kRingOff + kRing * kRawSlot;
    static constexpr uint32_t kBarOff = kTableOff + kRing * kBN * 4u;
    static constexpr uint32_t kNumBars = 2 * kPairStages + 2 * kRing + 1 + 4;
    static constexpr uint32_t kTotal = kBarOff + kNumBars * 8u + 16u;
};
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of `addr` (a shared::cta address of this CTA) in the CTA of rank `rank`
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool pf_mbar_wait_cluster(uint32_t bar, uint32_t parity)     // sees arrivals from the peer CTA
{
#pragma unroll 1
    for (uint32_t i = 0; i < kPfWaitLimit; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ void cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive, in BOTH CTAs of the pair, on the barrier at this shared-memory offset once every MMA issued so far is complete.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar)
{
    const unsigned short mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
                 "h"(mask)
                 : "memory");
}
// TMA tensor copy into this CTA's shared memory that completes on a barrier of either CTA of the pair (no multicast)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t cluster_bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(cluster_bar)
        : "memory");
}

// Grid: 1-D, clusters of two consecutive CTAs.  t CTAs first (pairs: 256 tokens x 256 rank rows),
// then main CTAs (pairs: 256 tokens x 256 features; a padding CTA past the last feature tile
// computes zeros and stores nothing).  Maps as for prefill_kernel, except that the boxes of xmap
// hold 128 token rows.
template <int BITS, typename T>
__global__ void __launch_bounds__(kPfThreads, 1)
prefill_pair_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap wmap,
               const __grid_constant__ CUtensorMap amap, const __grid_constant__ CUtensorMap bmap,
               const __grid_constant__ CUtensorMap ymap, const PrefillParams p)
{
    using L = PairSmem;
    constexpr int TOK = 256;                                    // tokens of the pair's tile; this CTA stages 128 of them
    constexpr int kStages = kPairStages;                        // (shadows the single-CTA kernel's depth)
    constexpr uint32_t kXBytes = L::kXBytes, kStageBytes = L::kStageBytes;
    const uint32_t cr = cluster_ctarank();                      // 0: leader (issues the MMAs), 1: peer
    constexpr int WPG = (BITS == 4) ? 16 : 12;                  // packed words per row and group
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = pf_smem_u32(smem);
    if (sbase & 1023u) {                                        // swizzle atoms need a 1024-byte aligned base
        if (threadIdx.x == 0) atomicExch(p.status, (int)FBQ_ERR_CUDA);
        return;
    }
    const uint32_t full0 = sbase + L::kBarOff, empty0 = full0 + 8u * kStages, rfull0 = empty0 + 8u * kStages,
                   rempty0 = rfull0 + 8u * kRing, done_bar = rempty0 + 8u * kRing, epi0 = done_bar + 8u;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + L::kBarOff + L::kNumBars * 8u);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool t_role = (int)blockIdx.x < p.n_t;                // t CTA or main CTA
    int m_tile, n_tile;
    if (t_role) {
        m_tile = (int)blockIdx.x / p.rt;
        n_tile = (int)blockIdx.x % p.rt;                        // tile of rank rows of A
    } else {
        m_tile = ((int)blockIdx.x - p.n_t) / p.nt;
        n_tile = ((int)blockIdx.x - p.n_t) % p.nt;
    }
    const int m0 = m_tile * TOK, n0 = n_tile * kBN;
    const int mh = m0 + 128 * (int)cr;                          // first token of the half this CTA stages
    const int nkb = t_role ? p.kb_main : p.kb_main + p.kb_slab;
    const int kb_x = p.kb_main;                                 // blocks below kb_x take their tokens from x

    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) {
            pf_mbar_init(full0 + 8u * i, t_role ? 1 : 17);      // leader's TMA lane + 8 producer warps of each CTA
            pf_mbar_init(empty0 + 8u * i, 1);
        }
        for (int i = 0; i < kRing; ++i) {
            pf_mbar_init(rfull0 + 8u * i, 2);                   // the two ring warps
            pf_mbar_init(rempty0 + 8u * i, kHalf / 32);         // a group is consumed by one half of the producers (8 warps)
        }
        pf_mbar_init(done_bar, 1);
        for (int i = 0; i < 4; ++i) pf_mbar_init(epi0 + 8u * i, 128);     // the four warps of a column quarter
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kMmaWarp) {                  // the MMA warp owns the tensor-memory allocation
        // the MMA warps of both CTAs of the pair allocate together (same columns in both)
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(pf_smem_u32(tmem_slot)),
                     "r"((uint32_t)TOK)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        tc_fence_before();
    }
    if (warp == kTmaWarp && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&xmap)) : "memory");
        if (t_role) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&amap)) : "memory");
        } else {
            if (p.rank > 0) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&bmap)) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&ymap)) : "memory");
        }
    }
    if (warp == kRawWarp && lane == 0)
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&wmap)) : "memory");
    cluster_sync();                          // barriers of both CTAs are initialised before anything arrives on them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp < kMmaWarp) {
        bool dead = false;
        if (!t_role) {
            // =================================================== producers
            // Half h of the warps takes the groups g = h, h+2, ... (K blocks 2g and 2g+1, stages 2h
            // and 2h+1); thread (row r, part) dequantises the codes [32*part, +32) of both blocks.
            const int h = warp >> 3, part = (warp >> 2) & 1, r = tid & 127;
            const bool row_ok = n0 + r < p.N;
            const int groups = p.kb_main >> 1;
            // this thread's words inside a ring slot: block b holds codes [64b, 64b+64) of the group
            uint32_t roff0, roff1;
            if (BITS == 4) {                                // 64-byte rows, 16-byte chunk c stored at c ^ ((row / 2) % 4)
                const uint32_t sw = (uint32_t)(r >> 1) & 3u;
                roff0 = (uint32_t)r * 64u + ((((uint32_t)part) ^ sw) << 4);
                roff1 = (uint32_t)r * 64u + ((((uint32_t)part + 2u) ^ sw) << 4);
            } else {                                        // 48-byte rows of four 12-byte runs
                roff0 = (uint32_t)r * 48u + (uint32_t)part * 12u;
                roff1 = roff0 + 24u;
            }
            const uint32_t ring0 = sbase + L::kRingOff, table0 = sbase + L::kTableOff + (uint32_t)r * 4u;
            // weight tile rows are 128 bytes (64 elements); the 16-byte chunk c of row r sits at c ^ (r % 8)
            const uint32_t wdst = sbase + kXBytes + (uint32_t)r * 128u;
            const uint32_t wsw = (uint32_t)r & 7u;
            const uint32_t lfull0 = mapa_shared(full0, 0);     // the leader's "full" barriers, as seen from this CTA
            uint32_t slot = (uint32_t)h, rphase = 0u;
#pragma unroll 1
            for (int g = h; g < groups; g += 2) {
                if (!pf_mbar_wait(rfull0 + 8u * slot, rphase)) { dead = true; break; }
                constexpr int NW = (BITS == 4) ? 4 : 3;
                uint32_t w[2][NW];
                const uint32_t rs = ring0 + slot * kRawSlot;
                if (BITS == 4) {
                    const uint4 a = lds128(rs + roff0), b = lds128(rs + roff1);
                    w[0][0] = a.x; w[0][1] = a.y; w[0][2] = a.z; w[0][NW - 1] = a.w;
                    w[1][0] = b.x; w[1][1] = b.y; w[1][2] = b.z; w[1][NW - 1] = b.w;
                } else {
#pragma unroll
                    for (int c = 0; c < 3; ++c) {
                        w[0][c] = lds32(rs + roff0 + 4u * c);
                        w[1][c] = lds32(rs + roff1 + 4u * c);
                    }
                }
                const uint32_t sz = lds32(table0 + slot * (kBN * 4u));      // s | z << 16 of (row, group)
                __syncwarp();
                if (lane == 0) pf_mbar_arrive(rempty0 + 8u * slot);   // the warp's words are in registers: the slot may be refilled
                slot += 2u;
                if (slot >= (uint32_t)kRing) { slot -= (uint32_t)kRing; rphase ^= 1u; }
                const float sc = __half2float(__ushort_as_half((unsigned short)(sz & 0xFFFFu)));
                const float ze = __half2float(__ushort_as_half((unsigned short)(sz >> 16)));
#pragma unroll
                for (int b = 0; b < 2; ++b) {
                    const int i = 2 * g + b, s = i % kStages;
                    if (i >= kStages && !pf_mbar_wait(empty0 + 8u * s, (uint32_t)(i / kStages - 1) & 1u)) { dead = true; break; }
                    uint32_t wb[16];
                    if (row_ok) {
                        uint32_t d[16];
                        Dequant<BITS, T>::run(w[b], sc, ze, d);
                        natural_pairs<BITS>(d, wb);
                    } else {
#pragma unroll
                        for (int c = 0; c < 16; ++c) wb[c] = 0u;
                    }
#pragma unroll
                    for (int kc = 0; kc < 4; ++kc)
                        sts128(wdst + (uint32_t)s * kStageBytes + ((((uint32_t)(4 * part + kc)) ^ wsw) << 4), wb[4 * kc], wb[4 * kc + 1], wb[4 * kc + 2],
                               wb[4 * kc + 3]);
                    pf_fence_proxy_async();                 // generic-proxy stores -> visible to the MMA's reads
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(lfull0 + 8u * s);       // one arrival per warp, on the leader's barrier
                }
                if (dead) break;
            }
            // ---- sub-branch blocks: token operand = t (fp32 scratch, rounded once); B arrives by TMA.
            // The halves take them in turn, one token row per thread.
            bool t_ready = false;
#pragma unroll 1
            for (int i = p.kb_main + h; i < nkb && !dead; i += 2) {
                const int s = i % kStages;
                if (i >= kStages && !pf_mbar_wait(empty0 + 8u * s, (uint32_t)(i / kStages - 1) & 1u)) { dead = true; break; }
                if (!t_ready) {                              // every warp of every t CTA of this token tile has stored its part
                    int seen = 0;
                    if (lane == 0) {
                        const int *flag = p.tflag + m_tile;
                        const int target = 16 * p.rt;
#pragma unroll 1
                        for (uint32_t spin = 0; spin < p.flag_polls; ++spin) {
                            asm volatile("ld.acquire.gpu.global.b32 %0, [%1];" : "=r"(seen) : "l"(flag) : "memory");
                            if (seen >= target) break;
                            __nanosleep(256);
                        }
                        seen = seen >= target;
                    }
                    t_ready = __shfl_sync(0xffffffffu, seen, 0) != 0;
                    if (!t_ready) { dead = true; break; }
                }
                const int j0 = (i - p.kb_main) * kBK;
                const int rr = tid & (kHalf - 1);            // token row of this CTA's half of the tile
                if (rr < 128) {
                    const int m = mh + rr;
                    uint32_t xa[32];
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        float4 t0 = make_float4(0.f, 0.f, 0.f, 0.f), t1 = t0;
                        if (m < p.M && j0 + 8 * c < p.rank) {              // rank is a multiple of 8: whole chunks
                            const float4 *ts = reinterpret_cast<const float4 *>(p.t32 + (size_t)m * p.rank + j0 + 8 * c);
                            t0 = __ldcg(ts);
                            t1 = __ldcg(ts + 1);
                        }
                        xa[4 * c] = P2<T>::pack(t0.x, t0.y); xa[4 * c + 1] = P2<T>::pack(t0.z, t0.w);
                        xa[4 * c + 2] = P2<T>::pack(t1.x, t1.y); xa[4 * c + 3] = P2<T>::pack(t1.z, t1.w);
                    }
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        sts128(sbase + (uint32_t)s * kStageBytes + (uint32_t)rr * 128u + ((((uint32_t)c) ^ ((uint32_t)rr & 7u)) << 4), xa[4 * c],
                               xa[4 * c + 1], xa[4 * c + 2], xa[4 * c + 3]);
                }
                pf_fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(lfull0 + 8u * s);
            }
            if (dead) {
                *abort_flag = 1;
                atomicExch(p.status, (int)FBQ_ERR_TIMEOUT);
            }
        }

        // =================================================== epilogue (same sixteen warps)
        // TMEM lane = weight row of the tile, column = token.  Warp w reads lanes 32*(w%4)..+31
        // (the only ones it may address) and the quarter w/4 of the columns.  Mode 0 stages the
        // tile in shared memory as [token][128 features] (the operand stages are free by now) and
        // each column quarter leaves with one TMA tensor store, which also clips the ragged edges.
        if (!dead && nkb > 0 && pf_mbar_wait(done_bar, 0)) {
            tc_fence_after();
            const int q = warp & 3, cg = warp >> 2;
            const int nn = n0 + 32 * q + lane;              // output feature (mode 0) / rank index (mode 1)
            const int c_begin = cg * (TOK / 4);
            if (m0 + c_begin < p.M) {                       // uniform over the four warps of a column quarter
#pragma unroll 1
                for (int c = c_begin; c < c_begin + TOK / 4; c += 32) {
                    if (m0 + c >= p.M) break;               // warp-uniform
                    uint32_t v[32];
                    tc_ld32(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)c, v);
                    tc_wait_ld();
                    if (!t_role) {
                        unsigned short *sp = reinterpret_cast<unsigned short *>(smem + (size_t)c * (kBN * 2)) + 32 * q + lane;
#pragma unroll
                        for (int j = 0; j < 32; ++j) sp[j * kBN] = to_bits16<T>(__uint_as_float(v[j]));
                    } else {
                        if (nn < p.rank) {                   // 32 lanes = 32 consecutive rank indices: 128-byte stores
                            float *tp = p.t32 + (size_t)(m0 + c) * p.rank + nn;
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (m0 + c + j < p.M) __stcg(tp + (size_t)j * p.rank, __uint_as_float(v[j]));
                        }
                    }
                }
                if (!t_role) {
                    pf_fence_proxy_async();                 // staged tile -> visible to the TMA store
                    pf_mbar_arrive(epi0 + 8u * cg);
                    if (q == 0 && lane == 0 && n0 < p.N) {   // (a padding CTA past the last feature tile stores nothing)
                        if (pf_mbar_wait(epi0 + 8u * cg, 0)) {
                            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                                         ::"l"(reinterpret_cast<uint64_t>(&ymap)), "r"(n0), "r"(m0 + c_begin),
                                           "r"(sbase + (uint32_t)c_begin * (kBN * 2))
                                         : "memory");
                            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // smem may go once it has been read
                        } else {
                            atomicExch(p.status, (int)FBQ_ERR_TIMEOUT);
                        }
                    }
                }
            }
            if (t_role) {
                // this warp's part of t is stored: make it visible, then count the warp in
                __threadfence();
                __syncwarp();
                if (lane == 0 && !p.test_skip_flag) atomicAdd(p.tflag + m_tile, 1);
            } else if (p.rank > 0 && tid == 0) {
                // this CTA has consumed t (its MMAs are complete).  The last main CTA of the token
                // tile leaves the flag and the count at zero for the next call.
                if (atomicAdd(p.tdone + m_tile, 1) == p.nt - 1) {
                    atomicExch(p.tflag + m_tile, 0);
                    atomicExch(p.tdone + m_tile, 0);
                }
            }
        }
        tc_fence_before();
    } else if (warp == kMmaWarp) {
        // =================================================== MMA warp
        // one MMA of the pair: 256 weight rows (128 per CTA) x 256 tokens (128 staged by each CTA) x 16
        constexpr uint32_t idesc = (1u << 4) | (P2<T>::kFmt << 7) | (P2<T>::kFmt << 10) | ((uint32_t)(TOK >> 3) << 17) |
                                   ((uint32_t)((2 * kBN) >> 4) << 24);
        bool dead = false;
#pragma unroll 1
        for (int i = 0; i < nkb && !dead && cr == 0; ++i) {     // only the leader CTA issues
            const int s = i % kStages;
            if (lane == 0) {
                if (!pf_mbar_wait_cluster(full0 + 8u * s, (uint32_t)(i / kStages) & 1u) || *abort_flag) {
                    dead = true;
                } else {
                    tc_fence_after();
                    const uint32_t x_base = sbase + (uint32_t)s * kStageBytes, w_base = x_base + kXBytes;
                    // every operand tile is K-major with 128-byte rows and the 128-byte swizzle, whether it
                    // arrived by TMA or was written by the producers: 32 bytes per 16 elements of K inside a row
#pragma unroll
                    for (int j = 0; j < kBK / 16; ++j)
                        tc_mma_pair(tmem_base, make_desc(w_base + j * 32), make_desc(x_base + j * 32), idesc, (i > 0 || j > 0) ? 1u : 0u);
                    tc_commit_pair(empty0 + 8u * s);         // the stage is free, in both CTAs, once these MMAs have read it
                }
            }
            dead = __shfl_sync(0xffffffffu, (int)dead, 0) != 0;
        }
        if (lane == 0) {
            if (dead) {
                *abort_flag = 1;
                atomicExch(p.status, (int)FBQ_ERR_TIMEOUT);
            } else if (nkb > 0 && cr == 0) {
                tc_commit_pair(done_bar);                    // accumulators complete in both CTAs
            }
        }
        __syncwarp();
        tc_fence_before();
    } else if (warp == kTmaWarp) {
        // =================================================== operand-stage copies
        if (lane == 0) {
            bool dead = false;
#pragma unroll 1
            for (int i = 0; i < nkb; ++i) {
                const int kb = i, s = i % kStages;
                if ((i >= kStages && !pf_mbar_wait(empty0 + 8u * s, (uint32_t)(i / kStages - 1) & 1u)) || *abort_flag) {
                    dead = true;
                    break;
                }
                const uint32_t bar = full0 + 8u * s;
                const uint32_t xt = sbase + (uint32_t)s * kStageBytes, wt = xt + kXBytes;
                // every copy of the pair completes on the LEADER's barrier; the leader announces the bytes of both
                const uint32_t lbar = mapa_shared(bar, 0);
                if (t_role) {
                    if (cr == 0) pf_mbar_expect_tx(bar, 2u * (kXBytes + kWBytes));
                    tma_load_2d_pair(xt, &xmap, kb * kBK, mh, lbar);
                    tma_load_2d_pair(wt, &amap, kb * kBK, n0, lbar);      // rows of A
                } else if (kb < kb_x) {
                    if (cr == 0) pf_mbar_expect_tx(bar, 2u * kXBytes);
                    tma_load_2d_pair(xt, &xmap, kb * kBK, mh, lbar);
                } else {
                    if (cr == 0) pf_mbar_expect_tx(bar, 2u * kWBytes);
                    tma_load_2d_pair(wt, &bmap, (kb - p.kb_main) * kBK, n0, lbar);   // rows of B
                }
            }
            if (dead) {
                *abort_flag = 1;
                atomicExch(p.status, (int)FBQ_ERR_TIMEOUT);
                for (int i = 0; i < 64; ++i) __nanosleep(1000);   // let the copies in flight land before the CTA exits
            }
        }
        __syncwarp();
    } else if (!t_role) {
        // =================================================== ring of packed codes and (s, z) table
        // Two warps; lane l of ring warp v owns the tile rows 64v + l and 64v + l + 32.  Per chunk of
        // eight groups it reads the rows' scales and zero points with 16-byte loads (two aligned chunks of the flat row-major arrays
        // cover any eight consecutive values), realigns them in registers, and before each group's
        // copy writes that group's (s | z << 16) words next to the ring slot.
        const int G = p.K / kGroupFast, groups = p.kb_main >> 1;
        const size_t n_chunks = (size_t)p.N * G / 8;        // N is a multiple of 8
        const uint4 *s_arr = reinterpret_cast<const uint4 *>(p.scales), *z_arr = reinterpret_cast<const uint4 *>(p.zeros);
        const int v = warp - kRawWarp;
        size_t a0[2];                                       // aligned 16-byte chunk holding group 0 of the row
        uint32_t off[2];                                    // position of group 0 inside that chunk (0..7)
        bool ok[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const int n = n0 + 64 * v + lane + 32 * k;
            ok[k] = n < p.N;
            const size_t f = (size_t)(ok[k] ? n : 0) * G;
            a0[k] = f >> 3;
            off[k] = (uint32_t)f & 7u;
        }
        uint4 raw[2][2][2];                                 // [row][s|z][low|high chunk] of the next eight groups
        auto fetch = [&](int c) {
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const size_t a = a0[k] + (size_t)c;
                const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
                raw[k][0][0] = (ok[k] && a < n_chunks) ? __ldg(s_arr + a) : zero;
                raw[k][1][0] = (ok[k] && a < n_chunks) ? __ldg(z_arr + a) : zero;
                raw[k][0][1] = (ok[k] && a + 1 < n_chunks) ? __ldg(s_arr + a + 1) : zero;
                raw[k][1][1] = (ok[k] && a + 1 < n_chunks) ? __ldg(z_arr + a + 1) : zero;
            }
        };
        // eight consecutive fp16 values starting `o` values into the 16-value window (lo, hi), as 4 pair-words
        auto realign = [](const uint4 &lo, const uint4 &hi, uint32_t o, uint32_t (&out)[4]) {
            uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
            if (o & 2u) {
#pragma unroll
                for (int i = 0; i < 7; ++i) w[i] = w[i + 1];
            }
            if (o & 4u) {
#pragma unroll
                for (int i = 0; i < 5; ++i) w[i] = w[i + 2];
            }
#pragma unroll
            for (int t = 0; t < 4; ++t) out[t] = __funnelshift_r(w[t], w[t + 1], (o & 1u) * 16u);
        };
        bool dead = false;
        fetch(0);
        const uint32_t ring0 = sbase + L::kRingOff, table0 = sbase + L::kTableOff + (uint32_t)(64 * v + lane) * 4u;
#pragma unroll 1
        for (int c = 0; 8 * c < groups && !dead; ++c) {
            uint32_t sz[2][8];                              // (s | z << 16) of [row][group of this chunk]
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                uint32_t sp[4], zp[4];
                realign(raw[k][0][0], raw[k][0][1], off[k], sp);
                realign(raw[k][1][0], raw[k][1][1], off[k], zp);
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    sz[k][2 * t] = pf_prmt(sp[t], zp[t], 0x5410u);
                    sz[k][2 * t + 1] = pf_prmt(sp[t], zp[t], 0x7632u);
                }
            }
            if (8 * (c + 1) < groups) fetch(c + 1);
#pragma unroll
            for (int g8 = 0; g8 < 8; ++g8) {
                const int gi = 8 * c + g8;
                if (gi < groups && !dead) {
                    const uint32_t slot = (uint32_t)gi % kRing;
                    if (lane == 0 && ((gi >= kRing && !pf_mbar_wait(rempty0 + 8u * slot, (uint32_t)(gi / kRing - 1) & 1u)) || *abort_flag))
                        dead = true;
                    dead = __shfl_sync(0xffffffffu, (int)dead, 0) != 0;     // also orders the table writes after the wait
                    if (!dead) {
#pragma unroll
                        for (int k = 0; k < 2; ++k)
                            asm volatile("st.shared.b32 [%0], %1;" ::"r"(table0 + slot * (kBN * 4u) + 128u * k), "r"(sz[k][g8]) : "memory");
                        __syncwarp();
                        if (lane == 0) {
                            if (v == 0) {
                                pf_mbar_expect_tx(rfull0 + 8u * slot, (uint32_t)kBN * WPG * 4u);
                                tma_load_2d(ring0 + slot * kRawSlot, &wmap, gi * WPG, n0, rfull0 + 8u * slot);
                            } else {
                                pf_mbar_arrive(rfull0 + 8u * slot);
                            }
                        }
                    }
                }
            }
        }
        if (dead && lane == 0) {
            *abort_flag = 1;
            atomicExch(p.status, (int)FBQ_ERR_TIMEOUT);
            for (int i = 0; i < 64; ++i) __nanosleep(1000);
        }
        __syncwarp();
    }
    cluster_sync();                          // both CTAs are done with their tensor memory and with each other's barriers
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TOK) : "memory");
    }
}


int g_pf_pdl = 1;             // launch with programmatic stream serialisation (prefill_set_pdl)

template <int BITS, typename T, int TOK>
cudaError_t launch_kernel(const CUtensorMap &xmap, const CUtensorMap &wmap, const CUtensorMap &amap, const CUtensorMap &bmap,
                          const CUtensorMap &ymap, const CUtensorMap &tmap, const PrefillParams &p, unsigned grid, cudaStream_t s)
{
    auto kern = prefill_kernel<BITS, T, TOK>;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Smem<TOK>::kTotal);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kPfThreads);
    cfg.dynamicSmemBytes = Smem<TOK>::kTotal;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = g_pf_pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, xmap, wmap, amap, bmap, ymap, tmap, p);
}

template <int BITS, typename T>
cudaError_t launch_pair_kernel(const CUtensorMap &xmap, const CUtensorMap &wmap, const CUtensorMap &amap, const CUtensorMap &bmap,
                               const CUtensorMap &ymap, const PrefillParams &p, unsigned grid, cudaStream_t s)
{
    auto kern = prefill_pair_kernel<BITS, T>;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PairSmem::kTotal);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kPfThreads);
    cfg.dynamicSmemBytes = PairSmem::kTotal;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, xmap, wmap, amap, bmap, ymap, p);
}

int g_pair = 0;

// 2-D tensor map of a row-major matrix: `cols` elements per row (16- or 32-bit), `rows` rows,
// boxes of box_cols x box_rows.  Reads outside the matrix return zero.
cudaError_t make_map(CUtensorMap *map, const void *base, bool elem32, size_t cols, size_t rows, int box_cols, int box_rows,
                     CUtensorMapSwizzle swizzle)
{
    static PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess) return e;
        if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
        encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
    }
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * (elem32 ? 4 : 2)};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = encode(map, elem32 ? CU_TENSOR_MAP_DATA_TYPE_UINT32 : CU_TENSOR_MAP_DATA_TYPE_UINT16, 2,
                              const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// K splits of a main tile when all tokens fit one tile of 128: as many as keep the CTA count near the
// number of SMs, at most 8, at least 2 groups of K per split.
int g_pf_skip_flag = 0, g_pf_flag_polls = 0;      // test switches (prefill_set_test)
int g_split_mode = 1;     // 0: never split K, 1: only deep K (>= 8192), 2: whenever tiles are few
int prefill_splits(int N, int K)
{
    if (g_split_mode == 0 || (g_split_mode == 1 && K < 8192)) return 1;
    const int nt = (N + kBN - 1) / kBN, G = K / kGroupFast;
    int s = 148 / nt;
    if (s > 8) s = 8;
    if (s > G / 2) s = G / 2;
    return s < 1 ? 1 : s;
}

template <typename T, int TOK, bool PAIR>
cudaError_t run_prefill(const LinearArgs &a, Workspace &ws, cudaStream_t s, int *launches)
{
    PrefillParams p{};
    p.scales = a.scales;
    p.zeros = a.zeros;
    p.t32 = ws.t_gen;
    p.y = a.y;
    p.status = ws.counters + kCtrStatus;
    p.M = a.M; p.N = a.N; p.K = a.K; p.rank = a.rank;
    p.kb_main = a.K / kBK;
    p.kb_slab = (a.rank + kBK - 1) / kBK;
    const int mt = (a.M + TOK - 1) / TOK;
    p.nt = (a.N + kBN - 1) / kBN;
    p.rt = (a.rank + kBN - 1) / kBN;
    if (PAIR) {                                     // CTAs come in pairs: feature tiles and rank tiles padded to even counts
        p.nt = (p.nt + 1) & ~1;
        p.rt = (p.rt + 1) & ~1;
    }
    // Few tokens mean few tiles: split K so that about one CTA per SM has work (single-CTA kernel, one
    // token tile).  The same number of splits goes to the t CTAs, which are cheap.
    p.splitk = p.splitt = 1;
    if (!PAIR && TOK == 128 && mt == 1) {             // (the split epilogue is written for one 32-column chunk per warp)
        const int want = prefill_splits(a.N, a.K);
        p.splitk = want;
        p.splitt = (a.rank > 0) ? want : 1;
    }
    p.n_t = mt * p.rt * p.splitt;
    p.tflag = ws.counters + kPfCtrBase;
    p.tdone = p.tflag + mt;
    p.split_ctr = p.tdone + mt;
    p.part = ws.partial;
    p.flag_polls = g_pf_flag_polls > 0 ? (uint32_t)g_pf_flag_polls : kPfFlagPolls;
    p.test_skip_flag = g_pf_skip_flag;
    CUtensorMap xmap, qmap, amap, bmap, ymap;
    cudaError_t e;
    if ((e = make_map(&xmap, a.x, false, (size_t)a.K, (size_t)a.M, kBK, PAIR ? 128 : TOK, CU_TENSOR_MAP_SWIZZLE_128B)) != cudaSuccess)
        return e;
    const int wpg = (a.bits == 4) ? 16 : 12;
    if ((e = make_map(&qmap, a.qw, true, (size_t)(a.K / kGroupFast) * wpg, (size_t)a.N, wpg, kBN,
                      a.bits == 4 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE)) != cudaSuccess)
        return e;
    if ((e = make_map(&ymap, a.y, false, (size_t)a.N, (size_t)a.M, kBN, TOK / 4, CU_TENSOR_MAP_SWIZZLE_NONE)) != cudaSuccess) return e;
    amap = bmap = xmap;
    CUtensorMap tmap = xmap;
    p.t16 = nullptr;
    p.rank_pad = p.kb_slab * kBK;
    if (!PAIR && a.rank > 0 && p.splitt == 1) {
        // t goes from the t CTAs to the main CTAs in the activation type, laid out like x, behind the fp32 slices of t
        p.t16 = ws.t_gen + (((size_t)a.M * a.rank + 3) & ~(size_t)3);
        if ((e = make_map(&tmap, p.t16, false, (size_t)p.rank_pad, (size_t)a.M, kBK, TOK, CU_TENSOR_MAP_SWIZZLE_128B)) != cudaSuccess) return e;
    }
    if (a.rank > 0) {
        if ((e = make_map(&amap, a.A, false, (size_t)a.K, (size_t)a.rank, kBK, kBN, CU_TENSOR_MAP_SWIZZLE_128B)) != cudaSuccess) return e;
        if ((e = make_map(&bmap, a.B, false, (size_t)a.rank, (size_t)a.N, kBK, kBN, CU_TENSOR_MAP_SWIZZLE_128B)) != cudaSuccess) return e;
    }
    const unsigned grid = (unsigned)p.n_t + (unsigned)p.nt * (unsigned)mt * (unsigned)p.splitk;
    if (PAIR)
        e = (a.bits == 4) ? launch_pair_kernel<4, T>(xmap, qmap, amap, bmap, ymap, p, grid, s)
                          : launch_pair_kernel<3, T>(xmap, qmap, amap, bmap, ymap, p, grid, s);
    else
        e = (a.bits == 4) ? launch_kernel<4, T, TOK>(xmap, qmap, amap, bmap, ymap, tmap, p, grid, s)
                          : launch_kernel<3, T, TOK>(xmap, qmap, amap, bmap, ymap, tmap, p, grid, s);
    if (e == cudaSuccess) ++*launches;
    return e;
}

inline bool aligned16(const void *q) { return (reinterpret_cast<uintptr_t>(q) & 15u) == 0; }

}  // namespace

// 1: token tiles of 256 run on CTA pairs (cta_group::2); 0: single-CTA kernel
void prefill_set_pair(int on) { g_pair = on ? 1 : 0; }
void prefill_set_split(int mode) { g_split_mode = mode; }
void prefill_set_pdl(int on) { g_pf_pdl = on ? 1 : 0; }
void prefill_set_test(int skip_flag, int flag_polls)
{
    g_pf_skip_flag = skip_flag;
    g_pf_flag_polls = flag_polls;
}

bool prefill_supported(const LinearArgs &a)
{
    return a.group == kGroupFast && a.K % kGroupFast == 0 && a.rank % 8 == 0 && a.rank <= kMaxRank && a.N % 8 == 0 &&
           a.M >= 1 && a.M <= (1 << 22);
}

// Scratch the prefill path needs in the workspace for this call: counters (zero between calls), floats
// of t (one slice per K split), floats of fp32 partial tiles (K split only).
void prefill_workspace_need(const LinearArgs &a, int *counters, size_t *t_floats, size_t *partial_floats)
{
    const int nt = (a.N + kBN - 1) / kBN;
    const int mt128 = (a.M + 127) / 128;
    const int splits = (a.M <= 128) ? prefill_splits(a.N, a.K) : 1;
    *counters = kPfCtrBase + 2 * mt128 + nt * mt128 + 2;
    *t_floats = (size_t)a.M * a.rank * splits + 4 + (size_t)a.M * ((a.rank + 63) / 64 * 64) / 2;      // fp32 slices of t, then t in the activation type
    *partial_floats = (splits > 1) ? (size_t)nt * splits * kBN * 128 : 0;
}

// ws.t_gen must hold M x rank floats and ws.counters prefill_counters_need(M) ints (the caller
// grows them; new counters start at zero and the kernel leaves them at zero).
// Operands that are not 16-byte aligned are refused (the caller then takes the generic kernel).
cudaError_t launch_prefill(const LinearArgs &a, Workspace &ws, cudaStream_t s, int *launches)
{
    if (!prefill_supported(a)) return cudaErrorInvalidConfiguration;
    if (!aligned16(a.x) || !aligned16(a.y) || !aligned16(a.qw) || !aligned16(a.scales) || !aligned16(a.zeros) ||
        (a.rank > 0 && (!aligned16(a.A) || !aligned16(a.B))))
        return cudaErrorInvalidConfiguration;
    if (a.M <= 128)
        return a.bf16 ? run_prefill<__nv_bfloat16, 128, false>(a, ws, s, launches) : run_prefill<__half, 128, false>(a, ws, s, launches);
    if (g_pair)
        return a.bf16 ? run_prefill<__nv_bfloat16, 256, true>(a, ws, s, launches) : run_prefill<__half, 256, true>(a, ws, s, launches);
    return a.bf16 ? run_prefill<__nv_bfloat16, 256, false>(a, ws, s, launches) : run_prefill<__half, 256, false>(a, ws, s, launches);
}

}  // namespace fbq
