// Decode kernel (M <= 16) of the FBQuant linear, sm_100a.
//
// One launch computes  y = x.dequant(Q,s,z)^T + (x.A^T).B^T  (Algorithm 1 step 6
// of the paper).  The paper's own kernel (Section 4.3) fuses dequantisation, the
// main product and the up-projection and leaves the down-projection t = x.A^T in
// a second launch; here t is produced by the same launch, so a decode step costs
// one launch per linear and y is written exactly once.
//
// Work split.  The grid is n_t + R x SK CTAs, about two per SM.  K is cut into SK
// slices (SK = 1 unless the tables do not fit shared memory); the 16-row tiles
// are dealt out in equal contiguous ranges, and a CTA walks its range tile by
// tile ("segments").
//
// Warp roles of a main CTA.  A producer warp streams the packed codes of the
// range: one TMA tensor copy per stage (16 groups x 16 rows, landing as
// [group][row][48 or 64 bytes]; mbarrier completion) into a ring of stages.
// Eight compute warps share every stage, two groups each.  At M <= 2 (integer
// form) a code masked out of its word is an unsigned byte operand of the 8-bit
// integer MMA as it stands and x is held as three signed base-256 digits per
// group scale, one digit per spare MMA column; above that (16-bit form) the codes
// are expanded with the exponent trick ((w & mask) | 0x6400 is 1024+q in fp16) and
// contracted with x by m16n8k16 MMAs.  In both forms the group scale multiplies
// the partial sum once per group and the zero point enters as s*z*sum(x).  An
// epilogue warp adds the eight warps' partial tiles of every segment (fixed
// order), adds t.B^T (per tile on tensor cores where the rank allows), rounds
// and stores y.
//
// t = x.A^T is computed by the first n_t CTAs of the grid (tensor-core blocks of
// eight rows of A), which raise a flag when it is complete; the main CTAs wait
// for the flag (bounded) where they need t.  Without such CTAs (M > 4, several
// K slices) every CTA's epilogue warp contributes a share of t, tiles shared
// between K slices are combined through scratch (whoever arrives last
// finishes), and a tile that is complete before t is waits in a list and is, at
// worst, handed to the warp that completes t: then nothing spins on another
// CTA.  All waits are bounded.
#include <cuda.h>
#include <cudaTypedefs.h>

#include <cstdio>
#include <cstdlib>
#include <mutex>
#include <type_traits>
#include <vector>

#include "fbq_common.cuh"

#ifndef FBQ_NACC
#define FBQ_NACC 2
#endif
namespace fbq {
namespace {

constexpr int kCW = 8;                       // compute warps per CTA
constexpr int kProdWarp = kCW + 1;         // warp kCW is the epilogue warp
constexpr int kWarps = kCW + 2;
constexpr int kThreads = kWarps * 32;
constexpr int kTileRows = 16;
constexpr int kMaxSeg = 64;                  // segments (tiles touched) per CTA
constexpr int kNBufMax = 8;                  // segment partial buffers in flight, at most (p.nbuf of them are used)
constexpr int kTUnitK = 1024;                // k extent of one unit of the down-projection
constexpr int kTMmaMaxM = 4;                   // tokens up to which the down-projection of the light variant runs on tensor cores
constexpr int kAPitch = kTUnitK + 8;         // elements between units of A in shared memory: 16 bytes past a multiple of 128, so
                                             // that eight units read at the same k fall into different banks
constexpr uint32_t kWaitLimit = 1u << 22;
constexpr int kEarlyStages = 1;                // weight stages prefetched before x has been requested
constexpr int kTUnitsOneWarp = 10;             // (token, unit) pairs of the down-projection one warp takes by itself
constexpr int kI8MaxM = 2;                     // tokens of the integer form: 3 digits (and a spare column) each fill the MMA's 8 columns
constexpr int kTPolls = 64;                  // looks at the "t complete" flag before a finished tile is parked

// counters[] layout (ints) inside the per-stream scratch
constexpr int kCtrReady = 3, kCtrPendingN = 4, kCtrFirstTile = 8;

struct DecodeParams {
    const void *x;
    const uint8_t *qw;
    const __half *scales;
    const __half *zeros;
    const void *A;
    const void *B;
    void *y;
    float *partial;     // [NT][maxslots][M][16]
    float *t;           // [M][rank], zero on entry, zero again on exit
    int *ctr;           // counters, see above; all zero on entry and on exit
    int *status;        // word that receives FBQ_ERR_TIMEOUT when a bounded wait runs out
    int M, N, K, G, rank;
    int SK, R, NT, CHG, NS, nbuf;
    int maxslots;
    int t_target;       // number of CTAs that contribute to t
    int n_t;            // > 0: the first n_t CTAs of the grid compute t and nothing else; the others only read it
    int t_late;         // test switch: contribute to t after the main loop
    int vt;             // lanes per quad whose accumulators are exchanged (tokens 2tq, 2tq+1 valid)
    int x_pitch;        // elements per token in shared memory
    int stage_bytes;
    int meta_rows;      // rows of the shared-memory scale / zero tables
    int a_cap;          // units of A held in shared memory
    int b_cap_rows;     // rows of B held in shared memory (0: read B from global memory)
    int t_wait;         // 1: a finished tile may wait in its segment buffer for t (as long as nobody is held up)
    int ab_alias;       // 1: B takes the place of A (and of the staged x) once the epilogue warp has used them; it issues the copy
    int off_tab, off_def, off_meta, off_x, off_px, off_segbuf, off_A, off_B, off_t, off_ring;
    unsigned long long *trace;   // optional phase timestamps [cta][warp][16] (tuning aid), else NULL
};

// ---------------------------------------------------------------- PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
// Completed or not, without waiting at all.
__device__ __forceinline__ uint32_t mbar_test(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
// Loads through 32-bit shared-window addresses (no 64-bit address arithmetic in the inner loops).
__device__ __forceinline__ uint32_t lds_u32(uint32_t a)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint4 lds_v4(uint32_t a)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ float2 lds_f2(uint32_t a)
{
    float2 v;
    asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(a));
    return v;
}
// Bounded wait: returns false when the limit is hit (never spins forever).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
#pragma unroll 1
    for (uint32_t i = 0; i < kWaitLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// The same for the warps that wait most of the time (producer, epilogue): they back off between
// looks so that their polling does not take issue slots from the compute warps of their SM.
__device__ __forceinline__ bool mbar_wait_idle(uint32_t bar, uint32_t parity)
{
#pragma unroll 1
    for (uint32_t i = 0; i < kWaitLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        __nanosleep(100);
    }
    return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
// One box of a 3-D tensor map (coordinates: word in group, weight row, group) into shared memory.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
                 "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ uint32_t lop3_and_or(uint32_t a, uint32_t mask, uint32_t orv)
{
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(a), "r"(mask), "r"(orv));   // (a & mask) | orv
    return r;
}

template <typename T> struct Pk;   // packed-pair arithmetic on raw 32-bit registers
template <> struct Pk<__half> {
    static __device__ __forceinline__ uint32_t sub(uint32_t a, uint32_t b)
    {
        uint32_t r;
        asm("sub.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
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
    static __device__ __forceinline__ void mma(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
    {
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
            : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    }
    static __device__ __forceinline__ float2 to_float2(uint32_t v)
    {
        return __half22float2(*reinterpret_cast<__half2 *>(&v));
    }
};
template <> struct Pk<__nv_bfloat16> {
    static __device__ __forceinline__ uint32_t sub(uint32_t a, uint32_t b)
    {
        uint32_t r;
        asm("sub.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
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
    static __device__ __forceinline__ void mma(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
    {
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
            : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    }
    static __device__ __forceinline__ float2 to_float2(uint32_t v)
    {
        return __bfloat1622float2(*reinterpret_cast<__nv_bfloat162 *>(&v));
    }
};

// ------------------------------------------------------------------ unpackers
// run(words, h) fills h[0..15] with one lane's 32 codes of one weight row as
// packed 16-bit floats in "fragment order", using nothing but shifts and one
// LOP3 per pair: a code field sitting at bit 3f (or 4e) of a 16-bit half is
// OR-ed into the mantissa of MAGIC = 1024 (fp16) or 128 (bf16), which yields
//        MAGIC + c*q      with c = 2^(field offset)  (kDiv below).
//   INT4: h[4i+e]  = codes (8i+e , 8i+e+4)  of word i          (i = 0..3, e = 0..3)
//   INT3: h[5i+f]  = codes (10i+f, 10i+5+f) of word i          (i = 0..2, f = 0..4)
//         h[15]    = codes (30, 31)
// No arithmetic is spent on removing MAGIC, c or the zero point per element:
// x is stored in shared memory already divided by c (a power of two), so the
// MMA yields  sum_k x_k*q_k + sum_k (MAGIC/c_k)*x_k ; the second sum and
// sum_k x_k depend on the token and group only and are tabulated once per CTA
// (P and X0), and the group's value is  s*(mma - P) - (s*z)*X0.
template <int BITS, typename T> struct Unpack;

template <> struct Unpack<4, __half> {
    static constexpr int kWords = 4;
    static constexpr float kMagic = 1024.f;
    static __device__ __forceinline__ int div_log2(int c) { return ((c & 7) & 1) ? 4 : 0; }   // odd nibbles sit 4 bits up
    static __device__ __forceinline__ void run(const uint32_t *w, uint32_t *h)
    {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t a = w[i], b = w[i] >> 8;
            h[4 * i + 0] = lop3_and_or(a, 0x000F000Fu, 0x64006400u);
            h[4 * i + 1] = lop3_and_or(a, 0x00F000F0u, 0x64006400u);
            h[4 * i + 2] = lop3_and_or(b, 0x000F000Fu, 0x64006400u);
            h[4 * i + 3] = lop3_and_or(b, 0x00F000F0u, 0x64006400u);
        }
    }
};
template <> struct Unpack<4, __nv_bfloat16> {
    static constexpr int kWords = 4;
    static constexpr float kMagic = 128.f;                     // 0x4300 | q  is 128 + q in bf16 (7 mantissa bits)
    static __device__ __forceinline__ int div_log2(int) { return 0; }
    static __device__ __forceinline__ void run(const uint32_t *w, uint32_t *h)
    {
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) h[4 * i + e] = lop3_and_or(w[i] >> (4 * e), 0x000F000Fu, 0x43004300u);
    }
};
template <> struct Unpack<3, __half> {
    static constexpr int kWords = 3;
    static constexpr float kMagic = 1024.f;
    static __device__ __forceinline__ int div_log2(int c)
    {
        if (c >= 30) return 0;
        const int f = (c % 10) % 5;                             // fields 0,3: bit 0; 1,4: bit 3; 2: bit 6 (3,4 after >> 9)
        return (f == 2) ? 6 : ((f == 1 || f == 4) ? 3 : 0);
    }
    static __device__ __forceinline__ void run(const uint32_t *w, uint32_t *h)
    {
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            const uint32_t a = w[i], b = w[i] >> 9;
            h[5 * i + 0] = lop3_and_or(a, 0x00070007u, 0x64006400u);
            h[5 * i + 1] = lop3_and_or(a, 0x00380038u, 0x64006400u);
            h[5 * i + 2] = lop3_and_or(a, 0x01C001C0u, 0x64006400u);
            h[5 * i + 3] = lop3_and_or(b, 0x00070007u, 0x64006400u);
            h[5 * i + 4] = lop3_and_or(b, 0x00380038u, 0x64006400u);
        }
        uint32_t l = lop3_and_or(w[0] >> 15, 0x00010001u, 0x64006400u);
        l = lop3_and_or(w[1] >> 14, 0x00020002u, l);
        h[15] = lop3_and_or(w[2] >> 13, 0x00040004u, l);
    }
};
template <> struct Unpack<3, __nv_bfloat16> {
    static constexpr int kWords = 3;
    static constexpr float kMagic = 128.f;
    static __device__ __forceinline__ int div_log2(int c)
    {
        if (c >= 30) return 0;
        const int f = (c % 10) % 5;                             // shifts 0, 6, 12: fields 0,2,4 at bit 0; 1,3 at bit 3
        return (f == 1 || f == 3) ? 3 : 0;
    }
    static __device__ __forceinline__ void run(const uint32_t *w, uint32_t *h)
    {
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            const uint32_t a = w[i], b = w[i] >> 6, c = w[i] >> 12;
            h[5 * i + 0] = lop3_and_or(a, 0x00070007u, 0x43004300u);
            h[5 * i + 1] = lop3_and_or(a, 0x00380038u, 0x43004300u);
            h[5 * i + 2] = lop3_and_or(b, 0x00070007u, 0x43004300u);
            h[5 * i + 3] = lop3_and_or(b, 0x00380038u, 0x43004300u);
            h[5 * i + 4] = lop3_and_or(c, 0x00070007u, 0x43004300u);
        }
        uint32_t l = lop3_and_or(w[0] >> 15, 0x00010001u, 0x43004300u);
        l = lop3_and_or(w[1] >> 14, 0x00020002u, l);
        h[15] = lop3_and_or(w[2] >> 13, 0x00040004u, l);
    }
};

// Position of code c (0..31) of a lane's 32-code run inside the fragment order
// above: returns 2*h_index + (0 = low half, 1 = high half).
template <int BITS> __device__ __forceinline__ int frag_pos(int c)
{
    if (BITS == 4) {
        const int i = c >> 3, e8 = c & 7;
        return 2 * (4 * i + (e8 & 3)) + (e8 >> 2);
    }
    if (c >= 30) return 2 * 15 + (c - 30);
    const int i = c / 10, f = c - 10 * i;
    return (f < 5) ? 2 * (5 * i + f) : 2 * (5 * i + f - 5) + 1;
}
// ------------------------------------------------- integer form (M <= 2)
// A 3- or 4-bit code masked out of its word where it sits is already an unsigned
// byte q * 2^j (j = the field's offset inside its byte): an operand of the 8-bit
// integer MMA (m16n8k32, u8 x s8 -> s32) as it stands, four codes per register,
// with no magic constant, no zero-point arithmetic and at most one shift per word:
//   INT4 word i:  r[2i]   = w & 0x0F0F0F0F          codes 8i+0, 8i+2, 8i+4, 8i+6
//                 r[2i+1] = w & 0xF0F0F0F0          codes 8i+1, 8i+3, 8i+5, 8i+7   (x 16)
//   INT3 word i:  r[3i]   = w & 0x0E070E07          codes 10i+0, 10i+3 (x 2), 10i+5, 10i+8 (x 2)
//                 r[3i+1] = w & 0x70387038          codes 10i+1 (x 8), 10i+4 (x 16), 10i+6 (x 8), 10i+9 (x 16)
//                 r[3i+2] = (w >> 6) & 0x02070207   codes 10i+2, bit i of code 30 (x 2), 10i+7, bit i of code 31 (x 2)
// The three bits of the bit-sliced codes 30 and 31 are three operands of their
// own, so a lane's 32 codes of INT3 take 36 slots (9 registers, 4.5 MMAs).
// x becomes fixed point: per group the power of two 2^e that puts the group's
// largest |x| into [2^20, 2^21) (the slots of the bit-sliced codes take up to 2x, and
// three signed digits hold |X| < 2^23 - 2^15), per slot X = rint(x 2^e 2^-j) (the slot's
// factor undone), and X is written with three signed base-256 digits, X = d0 2^16 +
// d1 2^8 + d2 (the bytes of (X + 0x808080) ^ 0x808080).  At M <= 2 the MMA has
// columns to spare: column 4m + i carries digit i of token m, the int32 sums of
// the three columns are exact, and they are added with the weights 2^16, 2^8, 1
// (times 2^-e) in fp32.  An fp16 or bf16 x is represented to 2^-17 of the
// group's maximum or better, far below the rounding of the fp16 product path.
template <int BITS> struct SlotsI8 {
    static constexpr int kRegs = (BITS == 4) ? 8 : 9;
    // code (0..31) of a lane's run whose value sits in byte j of register R
    static __host__ __device__ constexpr int code(int R, int j)
    {
        if (BITS == 4) return 8 * (R >> 1) + 2 * j + (R & 1);
        const int i = R / 3, f = R % 3;
        if (f == 2 && (j & 1)) return 30 + (j >> 1);
        return 10 * i + 5 * (j >> 1) + f + 3 * (j & 1);
    }
    // log2 of the factor x is stored with in that slot
    static __host__ __device__ constexpr int scale_log2(int R, int j)
    {
        if (BITS == 4) return (R & 1) ? -4 : 0;
        const int i = R / 3, f = R % 3;
        if (f == 2) return (j & 1) ? i - 1 : 0;
        if (f == 1) return (j & 1) ? -4 : -3;
        return (j & 1) ? -1 : 0;
    }
    static __device__ __forceinline__ void run(const uint32_t *w, uint32_t *r)
    {
        if (BITS == 4) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                r[2 * i] = w[i] & 0x0F0F0F0Fu;
                r[2 * i + 1] = w[i] & 0xF0F0F0F0u;
            }
        } else {
#pragma unroll
            for (int i = 0; i < 3; ++i) {
                r[3 * i] = w[i] & 0x0E070E07u;
                r[3 * i + 1] = w[i] & 0x70387038u;
                r[3 * i + 2] = (w[i] >> 6) & 0x02070207u;
            }
        }
    }
};
__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// x in shared memory: per token and 128-element group, 16-byte units are laid out
// [h_index / 4][lane t][h_index % 4], so that one 128-bit load per lane fetches the
// operands of two MMAs, conflict free.

__device__ __forceinline__ float ld_cg_f32(const float *p) { return __ldcg(p); }
__device__ __forceinline__ int ld_acquire(const int *p)
{
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void named_barrier_sync(int id, int nthreads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
// Tuning aid: SM cycle counter of this warp at a phase (cheap to read, unlike %globaltimer).
// Slot 15 of warp 0 additionally holds the global timer at kernel entry, to line CTAs up.
__device__ __forceinline__ void trace_mark(const DecodeParams &p, int slot)
{
    if (p.trace && (threadIdx.x & 31) == 0) {
        unsigned long long *row = p.trace + ((size_t)blockIdx.x * kWarps + (threadIdx.x >> 5)) * 16;
        row[slot] = (unsigned long long)clock64();
        if (slot == 0 && threadIdx.x == 0) {
            unsigned long long t;
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
            row[15] = t;
        }
    }
}

// --------------------------------------------------------------- tile epilogue
// Finishes one 16-row tile: main-path sums (slot i of scratch for i != myslot,
// the staged sums of this warp for i == myslot; staged == nullptr: every slot
// from scratch; always added in slot order), plus the up-projection t.B^T, one
// rounding, one store.  A lane handles (row, token) pairs idx = lane, lane+32, ..
// t comes from shared memory (s_t); B from shared memory when b_smem != nullptr
// (rows of this CTA's own tiles), else from global memory.  Kept out of line
// and free of unrolling on purpose: it runs once per tile, and the kernel's
// code must stay small enough for the instruction cache.
// (Arguments are passed one by one, not as the parameter struct, so that the call needs no
// stack.)  slots = scratch of this tile, Bg = B in global memory.
template <typename T>
__device__ __noinline__ void finish_tile(T *y, const float *slots, const T *Bg, int M, int N, int rank, int tile, int lane,
                                         const float *staged, int myslot, int cnt, const float *s_t, const T *b_smem)
{
    const size_t stride = (size_t)M * kTileRows;
#pragma unroll 1
    for (int idx = lane; idx < kTileRows * M; idx += 32) {
        const int row = idx & (kTileRows - 1), m = idx >> 4, n = tile * kTileRows + row;
        if (n >= N) continue;
        float v = 0.f;
#pragma unroll 1
        for (int i = 0; i < cnt; ++i) v += (staged && i == myslot) ? staged[idx] : ld_cg_f32(slots + i * stride + idx);
        if (rank > 0) {
            const float4 *trow = reinterpret_cast<const float4 *>(s_t + (size_t)m * rank);
            const uint4 *brow = b_smem ? reinterpret_cast<const uint4 *>(b_smem + (size_t)row * rank)
                                       : reinterpret_cast<const uint4 *>(Bg + (size_t)n * rank);
            float sub = 0.f;
#pragma unroll 2
            for (int c = 0; c < rank / 8; ++c) {
                const uint4 bv = brow[c];
                const float4 t0 = trow[2 * c], t1 = trow[2 * c + 1];
                const float2 b0 = Pk<T>::to_float2(bv.x), b1 = Pk<T>::to_float2(bv.y);
                const float2 b2 = Pk<T>::to_float2(bv.z), b3 = Pk<T>::to_float2(bv.w);
                sub = fmaf(t0.x, b0.x, sub); sub = fmaf(t0.y, b0.y, sub);
                sub = fmaf(t0.z, b1.x, sub); sub = fmaf(t0.w, b1.y, sub);
                sub = fmaf(t1.x, b2.x, sub); sub = fmaf(t1.y, b2.y, sub);
                sub = fmaf(t1.z, b3.x, sub); sub = fmaf(t1.w, b3.y, sub);
            }
            v += sub;
        }
        y[(size_t)m * N + n] = ActTraits<T>::from_float(v);
    }
}

// Claim a parked tile (exactly one claimant wins).
__device__ __forceinline__ bool tile_claim(const DecodeParams &p, int tile, int lane)
{
    int won = 0;
    if (lane == 0) won = (atomicAdd(p.ctr + kCtrFirstTile + tile, 1 << 16) < (1 << 16));
    return __shfl_sync(0xffffffffu, won, 0) != 0;
}

// --------------------------------------------------------------------- kernel
// The whole CTA program; `cta` is the CTA's index among the p.R * p.SK CTAs of its problem.
// HEAVY selects the variant for a heavy sub-branch (rank above 64, or many (token, unit) pairs of the
// down-projection per CTA): its units are shared by the eight compute warps and the tile finish
// keeps twice as many chunks of B in registers.  The light variant keeps both out of its code.
// Units of the down-projection (u = k chunk * rank + row of A) of CTA r out of R, for nkc chunks.  With
// at least as many CTAs as chunks, CTA r works on chunk r % nkc only (so it needs one chunk of x) and
// shares the chunk's rows evenly with the other CTAs of that chunk; with fewer CTAs the units are
// dealt out in contiguous ranges.  Host and device use the same function.
__host__ __device__ inline void unit_range(int r, int R, int rank, int nkc, int *u0, int *u1)
{
    if (rank <= 0 || nkc <= 0) {
        *u0 = *u1 = 0;
        return;
    }
    if (R >= nkc) {
        const int c = r % nkc, i = r / nkc, n_c = (R - c + nkc - 1) / nkc;      // CTAs of chunk c
        *u0 = c * rank + (int)((long long)i * rank / n_c);
        *u1 = c * rank + (int)((long long)(i + 1) * rank / n_c);
    } else {
        const long long TU = (long long)rank * nkc;
        *u0 = (int)((long long)r * TU / R);
        *u1 = (int)((long long)(r + 1) * TU / R);
    }
}

// A CTA that only computes t = x.A^T (the first n_t CTAs of a grid when the plan says so).  The main CTAs
// of one launch start over a span of time (they take SM slots as these become free), and a t that every
// CTA contributes to is complete only some microseconds after the LAST of them has started; these few
// CTAs are dispatched first, depend on nothing but x, and are done a few microseconds after the first.
// kTWarps warps each take blocks of up to eight rows of A of one 1024-wide k chunk: rows by bulk copies
// (requested before the wait on the previous kernel), the chunk of x by coalesced loads, then m16n8k16 MMAs
// whose rows are the tokens; fp32 atomics into t, and the last of these CTAs raises the "t complete" flag.
constexpr int kTWarps = 8;
constexpr int kTcK = 512;                     // k extent of a block of a t CTA
constexpr int kTcPitch = kTcK + 8;            // elements between rows in its shared memory (16 bytes past a multiple of 128)
template <typename T>
__device__ __noinline__ void t_cta_body(const DecodeParams &p, const int cta)
{
    extern __shared__ __align__(128) uint8_t smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tq = lane & 3;
    const uint32_t bar0 = smem_u32(smem);
    if (tid == 0) {
        for (int i = 0; i < kTWarps; ++i) mbar_init(bar0 + 8u * i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (warp >= kTWarps) {
        pdl_wait();
        pdl_launch_dependents();
        return;
    }
    const int area = (8 + p.M) * kTcPitch;                                     // elements per warp: 8 rows of A, M rows of x
    T *s_Aw = reinterpret_cast<T *>(smem + 1024) + (size_t)warp * area, *s_xw = s_Aw + 8 * kTcPitch;
    const uint32_t bar = bar0 + 8u * warp;
    const int bpr = (p.rank + 7) / 8, nkc = (p.K + kTcK - 1) / kTcK, nblocks = nkc * bpr;
    const T *A = static_cast<const T *>(p.A), *x = static_cast<const T *>(p.x);
    bool waited = false, dead = false;
    int round = 0;
#pragma unroll 1
    for (int b = cta * kTWarps + warp; b < nblocks; b += p.n_t * kTWarps, ++round) {
        const int kc = b / bpr, j0 = (b - kc * bpr) * 8, nrows = min(8, p.rank - j0);
        const int kbeg = kc * kTcK, nk = min(kTcK, p.K - kbeg);                // a multiple of 128
        __syncwarp();
        if (lane == 0) {
            if (round > 0) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the last block's reads are done
            mbar_expect_tx(bar, (uint32_t)(nrows * nk * 2));
        }
        __syncwarp();
        if (lane < nrows)
            bulk_g2s(smem_u32(s_Aw + (size_t)lane * kTcPitch), A + (size_t)(j0 + lane) * p.K + kbeg, (uint32_t)nk * 2u, bar);
        if (!waited) {                                                         // x may come from the previous kernel
            pdl_wait();
            pdl_launch_dependents();
            waited = true;
        }
#pragma unroll 1
        for (int m = 0; m < p.M; m += 2) {
            uint4 v[2][kTcK / 256];
#pragma unroll
            for (int mm = 0; mm < 2; ++mm)
#pragma unroll
                for (int i = 0; i < kTcK / 256; ++i) {
                    const int k = lane * 8 + 256 * i;
                    v[mm][i] = make_uint4(0u, 0u, 0u, 0u);
                    if (k < nk && m + mm < p.M) v[mm][i] = __ldcg(reinterpret_cast<const uint4 *>(x + (size_t)(m + mm) * p.K + kbeg + k));
                }
#pragma unroll
            for (int mm = 0; mm < 2; ++mm)
#pragma unroll
                for (int i = 0; i < kTcK / 256; ++i)
                    if (m + mm < p.M) *reinterpret_cast<uint4 *>(s_xw + (size_t)(m + mm) * kTcPitch + lane * 8 + 256 * i) = v[mm][i];
        }
        __syncwarp();
        if (!mbar_wait(bar, (uint32_t)round & 1u)) {
            dead = true;
            break;
        }
        const uint32_t *arow = reinterpret_cast<const uint32_t *>(s_Aw + (size_t)g * kTcPitch);
        const uint32_t *xa = reinterpret_cast<const uint32_t *>(s_xw + (size_t)g * kTcPitch);
        const bool col_ok = g < nrows, ra_ok = g < p.M;
        float d[4][4];
#pragma unroll
        for (int c = 0; c < 4; ++c) d[c][0] = d[c][1] = d[c][2] = d[c][3] = 0.f;
#pragma unroll 2
        for (int s16 = 0; s16 < nk / 16; s16 += 4) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int w = (s16 + c) * 8 + tq;                              // word index of k = 16 s + 2 tq
                uint32_t a[4] = {0u, 0u, 0u, 0u}, b0 = 0u, b1 = 0u;
                if (ra_ok) {
                    a[0] = xa[w];
                    a[2] = xa[w + 4];
                }
                if (col_ok) {
                    b0 = arow[w];
                    b1 = arow[w + 4];
                }
                Pk<T>::mma(d[c], a, b0, b1);
            }
        }
        const float v0 = (d[0][0] + d[1][0]) + (d[2][0] + d[3][0]), v1 = (d[0][1] + d[1][1]) + (d[2][1] + d[3][1]);
        const int c0 = 2 * tq;
        if (ra_ok) {
            if (c0 < nrows) atomicAdd(p.t + (size_t)g * p.rank + j0 + c0, v0);
            if (c0 + 1 < nrows) atomicAdd(p.t + (size_t)g * p.rank + j0 + c0 + 1, v1);
        }
    }
    if (!waited) {
        pdl_wait();
        pdl_launch_dependents();
    }
    if (dead && lane == 0) atomicExch(p.status, (int)FBQ_ERR_TIMEOUT);
    named_barrier_sync(2, kTWarps * 32);
    if (tid == 0) {
        __threadfence();
        if (atomicAdd(p.ctr + kCtrT, 1) == p.n_t - 1) {
            // all of t is in: publish it, then take part in the retire count like a finished tile would
            p.ctr[kCtrT] = 0;
            __threadfence();
            atomicExch(p.ctr + kCtrReady, 1);
            __threadfence();
            if (atomicAdd(p.ctr + kCtrDone, 1) + 1 == p.NT + 1) {
                __threadfence();
                for (int i = 0; i < 2 * p.NT; ++i) p.ctr[kCtrFirstTile + i] = 0;
                for (int i = 0; i < p.M * p.rank; ++i) p.t[i] = 0.f;
                p.ctr[kCtrDone] = 0;
                p.ctr[kCtrReady] = 0;
                p.ctr[kCtrPendingN] = 0;
            }
        }
    }
}

template <int BITS, typename T, int MT, bool HEAVY, bool I8>
__device__ __forceinline__ void decode_body(const DecodeParams &p, const CUtensorMap *wmap, const int cta_in_grid)
{
    if (cta_in_grid < p.n_t) {
        t_cta_body<T>(p, cta_in_grid);
        return;
    }
    const int cta = cta_in_grid - p.n_t;
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int GB = (BITS == 4) ? 64 : 48;          // packed bytes of one group of one row
    constexpr int NWORDS = Unpack<BITS, T>::kWords;    // words per lane per group
    // A stage in shared memory is [group][row][GB bytes], dense, as the tensor copy writes it: the
    // eight rows a warp reads at once are GB bytes apart, which spreads them over all banks (48 B:
    // 12 words, every lane of a 32-bit load in a bank of its own; 64 B: 128-bit loads, a quarter
    // warp covers 128 contiguous bytes).
    constexpr int NACC = FBQ_NACC;                     // independent MMA accumulator chains

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, tq = lane & 3;
    const int s = cta % p.SK, r = cta / p.SK;
    const int g0 = (int)((long long)s * p.G / p.SK), g1 = (int)((long long)(s + 1) * p.G / p.SK);
    const int ngs = g1 - g0;
    // whole 16-row tiles, dealt out in contiguous ranges; a "segment" is one tile of the range
    const int tile_first = (int)((long long)r * p.NT / p.R);
    const int nseg = (int)((long long)(r + 1) * p.NT / p.R) - tile_first;

    // units of the down-projection owned by this CTA: (row j of A, 1024-wide k chunk of the slice)
    const int kslice = ngs * kGroupFast;
    const int nkc = (kslice + kTUnitK - 1) / kTUnitK;
    int tu0, tu1;
    unit_range(r, p.R, p.rank, nkc, &tu0, &tu1);
    const bool has_t = (p.n_t == 0) && (p.rank > 0) && (tu1 > tu0);

    // shared memory: barriers | table | deferred list | meta | x | segbuf | A | B | t | ring
    trace_mark(p, 0);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem);
    const uint32_t st_full = smem_u32(bars), st_empty = st_full + 8u * p.NS;
    const uint32_t seg_full = st_empty + 8u * p.NS, seg_free = seg_full + 8u * kNBufMax;
    const uint32_t a_full = seg_free + 8u * kNBufMax, b_full = a_full + 8u, x_req = b_full + 8u, t_done = x_req + 8u;
    int *s_def = reinterpret_cast<int *>(smem + p.off_def);
    float2 *s_mf = reinterpret_cast<float2 *>(smem + p.off_meta);         // (s, s*z) [segment row][slice group]
    float2 *s_px = reinterpret_cast<float2 *>(smem + p.off_px);           // (P, X0)  [slice group][token]
    T *s_x = reinterpret_cast<T *>(smem + p.off_x);
    float *s_seg = reinterpret_cast<float *>(smem + p.off_segbuf);
    T *s_A = reinterpret_cast<T *>(smem + p.off_A);
    T *s_B = reinterpret_cast<T *>(smem + p.off_B);
    float *s_t = reinterpret_cast<float *>(smem + p.off_t);
    const int segbuf_floats = kCW * 8 * p.vt * 4 * MT;

    if (tid == 0) {
        for (int i = 0; i < p.NS; ++i) {
            mbar_init(st_full + 8u * i, 1);
            mbar_init(st_empty + 8u * i, kCW);
        }
        for (int i = 0; i < kNBufMax; ++i) {
            mbar_init(seg_full + 8u * i, kCW);
            mbar_init(seg_free + 8u * i, 1);
        }
        mbar_init(a_full, 1);
        mbar_init(b_full, 1);
        mbar_init(x_req, kCW);
        mbar_init(t_done, kCW);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    trace_mark(p, 1);

    const int b_rows = min(p.N, (tile_first + nseg) * kTileRows) - tile_first * kTileRows;   // weight rows of our tiles
    const bool b_in_smem = (p.rank > 0) && nseg > 0 && b_rows <= p.b_cap_rows;

    // This CTA's share of t = x.A^T:  t[m][j] += sum over its units (row j of A, k chunk of 1024);
    // units are numbered k-chunk-major (u = kc*rank + j).  A warp takes the units first, first +
    // stride, ...; a lane takes 8 elements out of every 256.  A comes from shared memory (bulk
    // copy) for the CTA's first a_cap units, else from global memory one unit ahead of use; x of a
    // (token, k chunk) is read from global memory once and kept in registers.  false = a wait ran out.
    auto t_units = [&](int first, int stride) -> bool {
        if (!mbar_wait(a_full, 0)) return false;
        const T *A = static_cast<const T *>(p.A);
        const T *x = static_cast<const T *>(p.x) + g0 * kGroupFast;
        auto load_a = [&](int u, uint4 (&av)[4]) {
            const int kc = u / p.rank, j = u - kc * p.rank;
            const int kbeg = kc * kTUnitK, nk = min(kTUnitK, kslice - kbeg);
            const bool in_smem = (u - tu0) < p.a_cap;
            const T *arow = in_smem ? s_A + (size_t)(u - tu0) * kAPitch : A + (size_t)j * p.K + g0 * kGroupFast + kbeg;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int k = lane * 8 + 256 * i;
                av[i] = make_uint4(0u, 0u, 0u, 0u);
                if (k < nk) av[i] = in_smem ? *reinterpret_cast<const uint4 *>(arow + k)
                                            : __ldg(reinterpret_cast<const uint4 *>(arow + k));
            }
        };
#pragma unroll 1
        for (int m = 0; m < p.M; ++m) {
            uint4 xv[4], an[4];
            int cur_kc = -1;
            if (first < tu1) load_a(first, an);
#pragma unroll 1
            for (int u = first; u < tu1; u += stride) {
                const int kc = u / p.rank;
                if (kc != cur_kc) {
                    cur_kc = kc;
                    const int kbeg = kc * kTUnitK, nk = min(kTUnitK, kslice - kbeg);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int k = lane * 8 + 256 * i;
                        xv[i] = make_uint4(0u, 0u, 0u, 0u);
                        if (k < nk) xv[i] = __ldcg(reinterpret_cast<const uint4 *>(x + (size_t)m * p.K + kbeg + k));
                    }
                }
                uint4 av[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) av[i] = an[i];
                if (u + stride < tu1) load_a(u + stride, an);       // the next row of A is in flight during the sum
                float v0 = 0.f, v1 = 0.f;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t aw[4] = {av[i].x, av[i].y, av[i].z, av[i].w};
                    const uint32_t xw[4] = {xv[i].x, xv[i].y, xv[i].z, xv[i].w};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float2 af = Pk<T>::to_float2(aw[q]), xf = Pk<T>::to_float2(xw[q]);
                        v0 = fmaf(xf.x, af.x, v0);
                        v1 = fmaf(xf.y, af.y, v1);
                    }
                }
                float v = v0 + v1;
                for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                if (lane == 0) atomicAdd(p.t + (size_t)m * p.rank + (u - kc * p.rank), v);
            }
        }
        return true;
    };

    // The same for the units of A that sit in shared memory, on the tensor cores: up to eight units of one
    // k chunk are the eight columns of m16n8k16 MMAs whose rows are the tokens (the chunk of x is staged
    // in shared memory first), four accumulators in turn.  One warp; far fewer
    // instructions and no long dependent chain, so t is complete soon after x is.
    auto t_units_mma = [&]() -> bool {
        if (p.M > kTMmaMaxM) return t_units(tu0, 1);
        if (!mbar_wait(a_full, 0)) return false;
        const int u_end = min(tu1, tu0 + p.a_cap);
        const T *x = static_cast<const T *>(p.x) + g0 * kGroupFast;
        T *s_xt = s_A + (size_t)p.a_cap * kAPitch;                              // x of the current k chunk, [token][kAPitch]
        int cur_kc = -1;
#pragma unroll 1
        for (int ub = tu0; ub < u_end;) {
            const int kc = ub / p.rank, j0 = ub - kc * p.rank;
            const int ue = min(min(ub + 8, u_end), (kc + 1) * p.rank);
            const int kbeg = kc * kTUnitK, nk = min(kTUnitK, kslice - kbeg);      // a multiple of 128
            if (kc != cur_kc) {
                // the chunk of x, coalesced and all loads in flight at once (two tokens at a time)
                cur_kc = kc;
                __syncwarp();
#pragma unroll 1
                for (int m = 0; m < p.M; m += 2) {
                    uint4 v[2][4];
#pragma unroll
                    for (int mm = 0; mm < 2; ++mm)
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int k = lane * 8 + 256 * i;
                            v[mm][i] = make_uint4(0u, 0u, 0u, 0u);
                            if (k < nk && m + mm < p.M) v[mm][i] = __ldcg(reinterpret_cast<const uint4 *>(x + (size_t)(m + mm) * p.K + kbeg + k));
                        }
#pragma unroll
                    for (int mm = 0; mm < 2; ++mm)
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            if (m + mm < p.M) *reinterpret_cast<uint4 *>(s_xt + (size_t)(m + mm) * kAPitch + lane * 8 + 256 * i) = v[mm][i];
                }
                __syncwarp();
            }
            const uint32_t *arow = reinterpret_cast<const uint32_t *>(s_A + (size_t)(ub - tu0 + g) * kAPitch);
            const uint32_t *xa = reinterpret_cast<const uint32_t *>(s_xt + (size_t)g * kAPitch);
            const bool col_ok = g < ue - ub, ra_ok = g < p.M;
            float d[4][4];
#pragma unroll
            for (int c = 0; c < 4; ++c) d[c][0] = d[c][1] = d[c][2] = d[c][3] = 0.f;
#pragma unroll 2
            for (int s16 = 0; s16 < nk / 16; s16 += 4) {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int w = (s16 + c) * 8 + tq;                          // word index of k = 16 s + 2 tq
                    uint32_t a[4] = {0u, 0u, 0u, 0u}, b0 = 0u, b1 = 0u;
                    if (ra_ok) {
                        a[0] = xa[w];
                        a[2] = xa[w + 4];
                    }
                    if (col_ok) {
                        b0 = arow[w];
                        b1 = arow[w + 4];
                    }
                    Pk<T>::mma(d[c], a, b0, b1);
                }
            }
            // d[.][0], d[.][1]: (token g, units 2 tq, 2 tq + 1) of the block (tokens 8.. do not occur here)
            const float v0 = (d[0][0] + d[1][0]) + (d[2][0] + d[3][0]), v1 = (d[0][1] + d[1][1]) + (d[2][1] + d[3][1]);
            const int c0 = 2 * tq, nb = ue - ub;
            if (ra_ok) {
                if (c0 < nb) atomicAdd(p.t + (size_t)g * p.rank + j0 + c0, v0);
                if (c0 + 1 < nb) atomicAdd(p.t + (size_t)g * p.rank + j0 + c0 + 1, v1);
            }
            ub = ue;
        }
        // units beyond the ones held in shared memory: the plain way
        if (u_end < tu1) return t_units(u_end, 1);
        return true;
    };

    // Who works the units off: the epilogue warp alone while there are few (token, unit) pairs (it has
    // nothing else to do until the first tile is through: light variant), all eight compute warps before
    // they turn to the weights when there are many (heavy variant: one warp would hold up the tiles).
    const bool t_by_compute = HEAVY && has_t && !p.t_late;

    if (warp == kProdWarp) {
        // =================================================== producer warp
        // A and B of this CTA (weights: independent of earlier kernels of the stream)
        if (has_t) {
            const T *A = static_cast<const T *>(p.A);
            const int na = min(tu1 - tu0, p.a_cap);
            uint32_t total = 0;
            for (int i = 0; i < na; ++i) {
                const int kc = (tu0 + i) / p.rank;               // units are numbered k-chunk-major: u = kc*rank + j
                total += (uint32_t)min(kTUnitK, kslice - kc * kTUnitK) * 2u;
            }
            if (lane == 0) mbar_expect_tx(a_full, total);
            __syncwarp();
            for (int i = lane; i < na; i += 32) {
                const int u = tu0 + i, kc = u / p.rank, j = u - kc * p.rank;
                const int nk = min(kTUnitK, kslice - kc * kTUnitK);
                bulk_g2s(smem_u32(s_A + (size_t)i * kAPitch), A + (size_t)j * p.K + g0 * kGroupFast + kc * kTUnitK,
                         (uint32_t)nk * 2u, a_full);
            }
        }
        if (b_in_smem && !p.ab_alias && lane == 0) {
            const uint32_t bytes = (uint32_t)b_rows * p.rank * 2u;
            mbar_expect_tx(b_full, bytes);
            bulk_g2s(smem_u32(s_B), static_cast<const T *>(p.B) + (size_t)tile_first * kTileRows * p.rank, bytes, b_full);
        }
        // the weight stream
        const uint32_t ring = smem_u32(smem + p.off_ring);
        int it = 0, slot = -1;
        uint32_t lap = 1u;                       // parity of the ring lap before the current one
        bool dead = false;
        for (int seg = 0; seg < nseg && !dead; ++seg) {
            const int tile = tile_first + seg;
            for (int pos = 0; pos < ngs; pos += p.CHG, ++it) {
                const int ng = min(p.CHG, ngs - pos);
                if (++slot == p.NS) {
                    slot = 0;
                    lap ^= 1u;
                }
                // Until the compute warps have put their loads of x (which everything waits for)
                // into the memory system, keep the prefetch shallow: x must not queue behind
                // megabytes of weights that cannot be used before it arrives.
                if (it == kEarlyStages && !mbar_wait(x_req, 0)) {
                    dead = true;
                    break;
                }
                if (it >= p.NS && !mbar_wait_idle(st_empty + 8u * slot, lap)) {
                    dead = true;
                    break;
                }
                // one box of CHG groups x 16 rows (rows past N and groups past G arrive as zeros; the
                // groups of a short last stage beyond ng are not used)
                if (lane == 0) {
                    mbar_expect_tx(st_full + 8u * slot, (uint32_t)p.stage_bytes);
                    tma_load_3d(ring + slot * p.stage_bytes, wmap, 0, tile * kTileRows, g0 + pos, st_full + 8u * slot);
                }
                __syncwarp();
            }
        }
        if (dead && lane == 0) atomicExch(p.status, (int)FBQ_ERR_TIMEOUT);
        trace_mark(p, 9);
        return;
    }

    if (warp < kCW) {
        // =================================================== compute warps
        // ---- fill shared memory.  The (s, s*z) table comes from weights, so its loads go out
        // before the wait on the previous kernel; x (divided by the field weights, permuted
        // into fragment order) and the per-group sums P, X0 after it.  All global loads of a
        // batch are issued before the first dependent instruction. ----
        const int nthr = kCW * 32;
        const int mpitch = ngs | 1;                  // odd pitch: the eight rows of a warp hit different banks
        {
            // (s, s*z) table: weights only, so it is filled before the wait on the previous kernel
            // (a warp per row, lanes over the row's groups: coalesced, and no division per entry)
            const uint16_t *sc = reinterpret_cast<const uint16_t *>(p.scales);
            const uint16_t *ze = reinterpret_cast<const uint16_t *>(p.zeros);
            const int nrows = nseg * kTileRows;
            // sixteen rows at a time, all their loads in flight before the first conversion
            constexpr int kRowsAtOnce = 16;
            for (int gl = lane; gl < ngs; gl += 32) {
#pragma unroll 1
                for (int row0 = warp; row0 < nrows; row0 += kRowsAtOnce * kCW) {
                    uint16_t sv[kRowsAtOnce], zv[kRowsAtOnce];
#pragma unroll
                    for (int u = 0; u < kRowsAtOnce; ++u) {
                        const int row = row0 + u * kCW;
                        const int n = min(tile_first * kTileRows + min(row, nrows - 1), p.N - 1);
                        const size_t mi = (size_t)n * p.G + g0 + gl;
                        sv[u] = sc[mi];
                        zv[u] = ze[mi];
                    }
#pragma unroll
                    for (int u = 0; u < kRowsAtOnce; ++u) {
                        const int row = row0 + u * kCW;
                        const float sf = __half2float(__ushort_as_half(sv[u]));
                        const float zf = __half2float(__ushort_as_half(zv[u]));
                        if (row < nrows) s_mf[row * mpitch + gl] = make_float2(sf, sf * zf);
                    }
                }
            }
        }

        // From here on x may come from the previous kernel of the stream.
        pdl_wait();
        pdl_launch_dependents();
        trace_mark(p, 3);
        if constexpr (I8) {
            // One lane takes one 32-element run of x (the k range of lane tq of one group), an even warp
            // the run's registers 0..3, an odd warp the rest.  Per group: 2^e puts the largest |x| into
            // [2^20, 2^21); per slot X = rint(x 2^e 2^-j) and its three signed base-256 digits.
            constexpr int NR = SlotsI8<BITS>::kRegs;
            const T *x = static_cast<const T *>(p.x);
            const int ncol = 3 * p.M;                                                 // three digit columns per token
            float2 *s_ux = reinterpret_cast<float2 *>(smem + p.off_px);               // (2^-e, X0) [slice group][token slot]
            uint4 *s_x8 = reinterpret_cast<uint4 *>(smem + p.off_x);                  // [slice group][chunk][column][lane tq]
            uint32_t *s_xt = reinterpret_cast<uint32_t *>(smem + p.off_x) + (size_t)ngs * 2 * ncol * 16;   // register 8
            if (p.M == 1)
                for (int i = tid; i < ngs; i += nthr) s_ux[2 * i + 1] = make_float2(0.f, 0.f);
            const int runs_per_tok = kslice / 32, nruns = p.M * runs_per_tok;         // multiples of 4
            const int upper = warp & 1;
            for (int base = 0; base < nruns; base += (kCW / 2) * 32) {
                const int idx = base + (warp >> 1) * 32 + lane;                       // whole quads are valid or not
                const bool valid = idx < nruns;
                const int m = valid ? idx / runs_per_tok : 0, run = valid ? idx - m * runs_per_tok : 0;
                uint4 xv[4];
                const uint4 *src = reinterpret_cast<const uint4 *>(x + (size_t)m * p.K + g0 * kGroupFast + run * 32);
#pragma unroll
                for (int i = 0; i < 4; ++i) xv[i] = valid ? __ldcg(src + i) : make_uint4(0u, 0u, 0u, 0u);
                if (base == 0) {                                  // our loads of x are on their way
                    __syncwarp();
                    if (lane == 0) mbar_arrive(x_req);
                }
                const uint16_t *e = reinterpret_cast<const uint16_t *>(xv);
                float xf[32];
                float amax = 0.f, xsum = 0.f;
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    T xe;
                    *reinterpret_cast<uint16_t *>(&xe) = e[c];
                    xf[c] = ActTraits<T>::to_float(xe);
                    amax = fmaxf(amax, fabsf(xf[c]));
                    xsum += xf[c];
                }
                // the four runs of one (token, group) sit in four consecutive lanes
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
                xsum += __shfl_xor_sync(0xffffffffu, xsum, 1);
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
                xsum += __shfl_xor_sync(0xffffffffu, xsum, 2);
                const uint32_t ex = min(max(__float_as_uint(amax) >> 23, 32u), 230u);          // biased exponent of the maximum
                const float xs = __uint_as_float((274u - ex) << 23);                         // 2^(20 - floor(log2 max))
                if (valid && !upper && (run & 3) == 0)
                    s_ux[(run >> 2) * 2 + m] = make_float2(__uint_as_float((ex - 20u) << 23), xsum);   // 1 / xs
                auto make = [&](auto rbeg, auto rend) {
                    constexpr int R0 = decltype(rbeg)::value, R1 = decltype(rend)::value;
                    uint32_t dg[R1 - R0][3];
#pragma unroll
                    for (int R = R0; R < R1; ++R) {
                        uint32_t y[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            constexpr float kPow[7] = {1.f / 16.f, 1.f / 8.f, 1.f / 4.f, 1.f / 2.f, 1.f, 2.f, 4.f};
                            const float f = xs * kPow[SlotsI8<BITS>::scale_log2(R, j) + 4];
                            const int X = __float2int_rn(xf[SlotsI8<BITS>::code(R, j)] * f);
                            y[j] = ((uint32_t)X + 0x00808080u) ^ 0x00808080u;
                        }
                        // digit i of the four slots -> one register (byte j = slot j)
                        const uint32_t lo01 = __byte_perm(y[0], y[1], 0x5140), lo23 = __byte_perm(y[2], y[3], 0x5140);   // b0 b0' b1 b1'
                        dg[R - R0][2] = __byte_perm(lo01, lo23, 0x5410);
                        dg[R - R0][1] = __byte_perm(lo01, lo23, 0x7632);
                        dg[R - R0][0] = __byte_perm(__byte_perm(y[0], y[1], 0x0062), __byte_perm(y[2], y[3], 0x0062), 0x5410);
                    }
                    if (valid) {
                        const int gl = run >> 2, lq = run & 3;
#pragma unroll
                        for (int k = 0; k < 3; ++k) {
                            const int col = 3 * m + k;
                            s_x8[(size_t)((gl * 2 + R0 / 4) * ncol + col) * 4 + lq] = make_uint4(dg[0][k], dg[1][k], dg[2][k], dg[3][k]);
                            if constexpr (R1 - R0 == 5) s_xt[(size_t)(gl * ncol + col) * 4 + lq] = dg[4][k];
                        }
                    }
                };
                if (!upper) make(std::integral_constant<int, 0>{}, std::integral_constant<int, 4>{});
                else make(std::integral_constant<int, 4>{}, std::integral_constant<int, NR>{});
            }
        } else {
            // One thread prepares one 32-element run of x: 64 contiguous bytes in, the run's 16
            // fragment-order pairs (four 16-byte units) out, with compile-time positions.
            const T *x = static_cast<const T *>(p.x);
            const int runs_per_tok = kslice / 32, nruns = p.M * runs_per_tok;     // multiples of 4
            const int mp = 8 * MT;                                                // token slots of the (P, X0) table
            for (int i = tid; i < ngs * mp; i += nthr)                            // tokens beyond M contribute nothing
                if (i % mp >= p.M) s_px[i] = make_float2(0.f, 0.f);
            for (int base = 0; base < nruns; base += nthr) {
                const int idx = base + tid;                                       // whole quads are valid or not
                const bool valid = idx < nruns;
                const int m = valid ? idx / runs_per_tok : 0, run = valid ? idx - m * runs_per_tok : 0;
                uint4 xv[4];
                const uint4 *src = reinterpret_cast<const uint4 *>(x + (size_t)m * p.K + g0 * kGroupFast + run * 32);
#pragma unroll
                for (int i = 0; i < 4; ++i) xv[i] = valid ? __ldcg(src + i) : make_uint4(0u, 0u, 0u, 0u);
                if (base == 0) {                                  // our loads of x are on their way
                    __syncwarp();
                    if (lane == 0) mbar_arrive(x_req);
                }
                const uint16_t *e = reinterpret_cast<const uint16_t *>(xv);
                uint32_t h[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) h[i] = 0u;
                float psum = 0.f, xsum = 0.f;
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    const int pos = frag_pos<BITS>(c);                            // folds to a constant
                    T xe;
                    *reinterpret_cast<uint16_t *>(&xe) = e[c];
                    const float xf = ActTraits<T>::to_float(xe);
                    // exact division by the field weight (a power of two; up to fp16 underflow).
                    // P is summed from the stored value, so the MMA's bias term cancels exactly.
                    const T xs = ActTraits<T>::from_float(ldexpf(xf, -Unpack<BITS, T>::div_log2(c)));
                    h[pos >> 1] |= (uint32_t)(*reinterpret_cast<const uint16_t *>(&xs)) << (16 * (pos & 1));
                    psum = fmaf(Unpack<BITS, T>::kMagic, ActTraits<T>::to_float(xs), psum);
                    xsum += xf;
                }
                if (valid) {
                    uint4 *dst = reinterpret_cast<uint4 *>(s_x + (size_t)m * p.x_pitch + (run >> 2) * kGroupFast);
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4)
                        dst[q4 * 4 + (run & 3)] = make_uint4(h[4 * q4], h[4 * q4 + 1], h[4 * q4 + 2], h[4 * q4 + 3]);
                }
                // the four runs of one (token, group) sit in four consecutive lanes
                psum += __shfl_xor_sync(0xffffffffu, psum, 1);
                xsum += __shfl_xor_sync(0xffffffffu, xsum, 1);
                psum += __shfl_xor_sync(0xffffffffu, psum, 2);
                xsum += __shfl_xor_sync(0xffffffffu, xsum, 2);
                if (valid && (run & 3) == 0) s_px[(run >> 2) * mp + m] = make_float2(psum, xsum);
            }
        }
        trace_mark(p, 4);
        bool dead = false;
        named_barrier_sync(1, kCW * 32);
        trace_mark(p, 5);
        if (t_by_compute) {
            if (!t_units(tu0 + warp, kCW)) dead = true;
            __threadfence();
            __syncwarp();
            if (lane == 0) mbar_arrive(t_done);
        }

        // ---- consumer: every stage is shared; this warp takes an eighth of its groups ----
        const uint8_t *ring_ptr = smem + p.off_ring;
        int it = 0, slot = -1;
        uint32_t lap = 1u;                       // parity of the current lap around the ring, inverted
        long long t_wait = 0;                    // trace: cycles spent waiting for weight stages
        for (int seg = 0; seg < nseg && !dead; ++seg) {
            float acc[MT][4];
            float accz[2] = {0.f, 0.f};          // integer form: sum of (s z) X0 of rows g and g + 8
#pragma unroll
            for (int b = 0; b < MT; ++b)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[b][i] = 0.f;
            if constexpr (I8) {
                // Integer form, written lean: everything that does not change per unit sits in registers as
                // 32-bit shared-memory addresses and strides, and nothing in the unit loop is conditional.
                // Lanes whose MMA column carries no digit (column 3 of a token, tokens >= M) read a column
                // that exists instead: their sums land in output columns nobody looks at.
                constexpr int NR = SlotsI8<BITS>::kRegs;
                const int ncol = 3 * p.M, CHG = p.CHG, NS = p.NS;
                const int cc = (g < 4 * p.M && (g & 3) != 3) ? g - (g >> 2) : 0;
                const uint32_t sbase = smem_u32(smem);
                const uint32_t x_gstride = (uint32_t)ncol * 128u, x_chunk1 = (uint32_t)ncol * 64u;
                const uint32_t x_lane = sbase + p.off_x + (uint32_t)(cc * 4 + tq) * 16u;
                const uint32_t xt_lane = sbase + p.off_x + (uint32_t)ngs * x_gstride + (uint32_t)(cc * 4 + tq) * 4u;
                const uint32_t xt_gstride = (uint32_t)ncol * 16u;
                const uint32_t ux_lane = sbase + p.off_px + (uint32_t)(tq >> 1) * 8u;
                const uint32_t w_lane = sbase + p.off_ring + (uint32_t)(g * GB + tq * (GB / 4));
                const uint32_t m_lane = sbase + p.off_meta + (uint32_t)((seg * kTileRows + g) * mpitch) * 8u;
                const uint32_t stage_bytes = (uint32_t)p.stage_bytes;
                for (int pos = 0; pos < ngs; pos += CHG, ++it) {
                    const int ng = min(CHG, ngs - pos);
                    if (++slot == NS) {
                        slot = 0;
                        lap ^= 1u;
                    }
                    if (!mbar_wait(st_full + 8u * slot, lap ^ 1u)) {
                        dead = true;
                        break;
                    }
                    const int gbeg = (warp * ng) >> 3, gend = ((warp + 1) * ng) >> 3;      // this warp's groups of the stage
                    uint32_t wa = w_lane + (uint32_t)slot * stage_bytes + (uint32_t)gbeg * (kTileRows * GB);
                    uint32_t xa = x_lane + (uint32_t)(pos + gbeg) * x_gstride;
                    uint32_t xta = xt_lane + (uint32_t)(pos + gbeg) * xt_gstride;
                    uint32_t ua = ux_lane + (uint32_t)(pos + gbeg) * 16u;
                    uint32_t ma = m_lane + (uint32_t)(pos + gbeg) * 8u;
#pragma unroll 1
                    for (int gi = gbeg; gi < gend; ++gi) {
                        uint32_t wra[NWORDS], wrb[NWORDS];
                        if constexpr (BITS == 4) {
                            const uint4 va = lds_v4(wa), vb = lds_v4(wa + 8 * GB);
                            wra[0] = va.x; wra[1] = va.y; wra[2] = va.z; wra[3] = va.w;
                            wrb[0] = vb.x; wrb[1] = vb.y; wrb[2] = vb.z; wrb[3] = vb.w;
                        } else {
#pragma unroll
                            for (int i = 0; i < NWORDS; ++i) {
                                wra[i] = lds_u32(wa + 4 * i);
                                wrb[i] = lds_u32(wa + 8 * GB + 4 * i);
                            }
                        }
                        const uint4 x0 = lds_v4(xa), x1 = lds_v4(xa + x_chunk1);
                        const float2 fa = lds_f2(ma), fb = lds_f2(ma + 8u * (uint32_t)mpitch * 8u), ux = lds_f2(ua);
                        uint32_t ra[NR], rb[NR];
                        SlotsI8<BITS>::run(wra, ra);
                        SlotsI8<BITS>::run(wrb, rb);
                        int d[4] = {0, 0, 0, 0};
                        mma_u8s8(d, ra[0], rb[0], ra[1], rb[1], x0.x, x0.y);
                        mma_u8s8(d, ra[2], rb[2], ra[3], rb[3], x0.z, x0.w);
                        mma_u8s8(d, ra[4], rb[4], ra[5], rb[5], x1.x, x1.y);
                        mma_u8s8(d, ra[6], rb[6], ra[7], rb[7], x1.z, x1.w);
                        if constexpr (BITS == 3) mma_u8s8(d, ra[NR - 1], rb[NR - 1], 0u, 0u, lds_u32(xta), 0u);
                        const float sa = fa.x * ux.x, sb = fb.x * ux.x;
                        acc[0][0] = fmaf(sa, (float)d[0], acc[0][0]);
                        acc[0][1] = fmaf(sa, (float)d[1], acc[0][1]);
                        acc[0][2] = fmaf(sb, (float)d[2], acc[0][2]);
                        acc[0][3] = fmaf(sb, (float)d[3], acc[0][3]);
                        accz[0] = fmaf(fa.y, ux.y, accz[0]);
                        accz[1] = fmaf(fb.y, ux.y, accz[1]);
                        wa += kTileRows * GB;
                        xa += x_gstride;
                        xta += xt_gstride;
                        ua += 16u;
                        ma += 8u;
                    }
                    // stage consumed by this warp
                    __syncwarp();
                    if (lane == 0) mbar_arrive(st_empty + 8u * slot);
                }
            } else
            for (int pos = 0; pos < ngs; pos += p.CHG, ++it) {
                const int ng = min(p.CHG, ngs - pos);
                if (++slot == p.NS) {
                    slot = 0;
                    lap ^= 1u;
                }
                const long long c_wait = p.trace ? clock64() : 0;
                if (!mbar_wait(st_full + 8u * slot, lap ^ 1u)) {
                    dead = true;
                    break;
                }
                if (p.trace) t_wait += clock64() - c_wait;
                if (it == 0) trace_mark(p, 6);
                const uint8_t *slot_ptr = ring_ptr + (size_t)slot * p.stage_bytes;
                const int gbeg = warp * ng / kCW, gend = (warp + 1) * ng / kCW;     // this warp's groups of the stage
                const float2 *meta_a = s_mf + (size_t)(seg * kTileRows + g) * mpitch + pos;   // row g; row g+8 is 8 rows on
                const float2 *meta_b = meta_a + 8 * mpitch;

                for (int gi = gbeg; gi < gend; ++gi) {
                    const float2 fa = meta_a[gi], fb = meta_b[gi];          // (s, s*z) of rows g and g+8
                    uint32_t wa[NWORDS], wb[NWORDS];
                    const uint8_t *pa = slot_ptr + gi * (kTileRows * GB) + g * GB + tq * (GB / 4);
                    const uint8_t *pb = pa + 8 * GB;
                    if constexpr (BITS == 4) {
                        const uint4 va = *reinterpret_cast<const uint4 *>(pa), vb = *reinterpret_cast<const uint4 *>(pb);
                        wa[0] = va.x; wa[1] = va.y; wa[2] = va.z; wa[3] = va.w;
                        wb[0] = vb.x; wb[1] = vb.y; wb[2] = vb.z; wb[3] = vb.w;
                    } else {
#pragma unroll
                        for (int i = 0; i < NWORDS; ++i) {
                            wa[i] = reinterpret_cast<const uint32_t *>(pa)[i];
                            wb[i] = reinterpret_cast<const uint32_t *>(pb)[i];
                        }
                    }
                    uint32_t ha[16], hb[16];
                    Unpack<BITS, T>::run(wa, ha);
                    Unpack<BITS, T>::run(wb, hb);

#pragma unroll
                    for (int b = 0; b < MT; ++b) {
                        // (P, X0) of tokens 8b+2tq and 8b+2tq+1 for this group; the chain starts at -P
                        const float4 px = *reinterpret_cast<const float4 *>(s_px + (size_t)(pos + gi) * (8 * MT) + 8 * b + 2 * tq);
                        float tmp[NACC][4];
#pragma unroll
                        for (int c = 0; c < NACC; ++c) tmp[c][0] = tmp[c][1] = tmp[c][2] = tmp[c][3] = 0.f;
                        tmp[0][0] = tmp[0][2] = -px.x;
                        tmp[0][1] = tmp[0][3] = -px.z;
                        const int token = 8 * b + g;
                        const uint4 *xg = reinterpret_cast<const uint4 *>(s_x + (size_t)token * p.x_pitch +
                                                                          (size_t)(pos + gi) * kGroupFast);
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            uint4 xv = make_uint4(0u, 0u, 0u, 0u);
                            if (token < p.M) xv = xg[q4 * 4 + tq];
                            const uint32_t a0[4] = {ha[4 * q4 + 0], hb[4 * q4 + 0], ha[4 * q4 + 1], hb[4 * q4 + 1]};
                            const uint32_t a1[4] = {ha[4 * q4 + 2], hb[4 * q4 + 2], ha[4 * q4 + 3], hb[4 * q4 + 3]};
                            Pk<T>::mma(tmp[q4 % NACC], a0, xv.x, xv.y);
                            Pk<T>::mma(tmp[q4 % NACC], a1, xv.z, xv.w);
                        }
                        float d[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            d[i] = tmp[0][i];
#pragma unroll
                            for (int c = 1; c < NACC; ++c) d[i] += tmp[c][i];
                        }
                        // s*(mma - P) - (s*z)*X0
                        acc[b][0] = fmaf(-fa.y, px.y, fmaf(fa.x, d[0], acc[b][0]));
                        acc[b][1] = fmaf(-fa.y, px.w, fmaf(fa.x, d[1], acc[b][1]));
                        acc[b][2] = fmaf(-fb.y, px.y, fmaf(fb.x, d[2], acc[b][2]));
                        acc[b][3] = fmaf(-fb.y, px.w, fmaf(fb.x, d[3], acc[b][3]));
                    }
                }
                // stage consumed by this warp
                __syncwarp();
                if (lane == 0) mbar_arrive(st_empty + 8u * slot);
            }
            if (dead) break;
            if constexpr (I8) {
                // Columns 4m, 4m+1, 4m+2 are the digits of token m (weights 2^16, 2^8, 1), column 4m+3 is empty;
                // lane tq = 2m holds the first two, 2m + 1 the rest; afterwards lane tq = 0 holds (token 0,
                // token 1) of rows g and g + 8.
                const float w0 = (tq & 1) ? 1.f : 65536.f, w1 = (tq & 1) ? 0.f : 256.f;
                float vg = fmaf(acc[0][1], w1, acc[0][0] * w0), vh = fmaf(acc[0][3], w1, acc[0][2] * w0);
                vg += __shfl_xor_sync(0xffffffffu, vg, 1);
                vh += __shfl_xor_sync(0xffffffffu, vh, 1);
                vg -= accz[0];
                vh -= accz[1];
                acc[0][0] = vg;
                acc[0][1] = __shfl_xor_sync(0xffffffffu, vg, 2);
                acc[0][2] = vh;
                acc[0][3] = __shfl_xor_sync(0xffffffffu, vh, 2);
            }

            // ---- deposit this warp's partial tile for the epilogue warp ---------------
            const int buf = seg % p.nbuf;
            if (seg >= p.nbuf && !mbar_wait(seg_free + 8u * buf, (uint32_t)(seg / p.nbuf - 1) & 1u)) {
                dead = true;
                break;
            }
            if (tq < p.vt) {
                float4 *dst = reinterpret_cast<float4 *>(s_seg + (size_t)buf * segbuf_floats +
                                                         (size_t)((warp * 8 + g) * p.vt + tq) * 4 * MT);
#pragma unroll
                for (int b = 0; b < MT; ++b) dst[b] = make_float4(acc[b][0], acc[b][1], acc[b][2], acc[b][3]);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(seg_full + 8u * buf);
            trace_mark(p, seg == 0 ? 7 : 8);
        }
        trace_mark(p, 9);
        if (p.trace && lane == 0) p.trace[((size_t)blockIdx.x * kWarps + warp) * 16 + 12] = (unsigned long long)t_wait;
        if (dead && lane == 0) atomicExch(p.status, (int)FBQ_ERR_TIMEOUT);
        return;
    }

    // ======================================================= epilogue warp
    pdl_wait();
    pdl_launch_dependents();
    trace_mark(p, 2);
    int n_retired = 0;          // tiles finished by this warp (+1 token if it completed t)
    int n_def = 0;              // tiles this warp must finish once t is complete (s_def[])
    bool t_local = (p.rank == 0);   // t is complete and copied to shared memory
    bool dead = false;
    float *s_stage = s_t + (size_t)p.M * p.rank;     // this warp's staged main sums [token][16]

    // Looks at the "t complete" flag; on the first sighting copies t to shared memory.
    auto t_poll = [&]() -> bool {
        if (t_local) return true;
        int ready = 0;
        if (lane == 0) ready = ld_acquire(p.ctr + kCtrReady);
        ready = __shfl_sync(0xffffffffu, ready, 0);
        if (!ready) return false;
        for (int i = lane; i < p.M * p.rank; i += 32) s_t[i] = ld_cg_f32(p.t + i);
        __syncwarp();
        t_local = true;
        return true;
    };
    auto own_b = [&](int tile) -> const T * {
        return (b_in_smem && tile >= tile_first && tile < tile_first + nseg)
                   ? s_B + (size_t)(tile - tile_first) * kTileRows * p.rank
                   : nullptr;
    };
    // Fast finish (rank <= 64, heavy variant 128; one K slice): lanes 2i and 2i+1 share row i of the tile; a lane holds
    // every other 8-element chunk of that row of B in registers, requested before the wait for the
    // segment, so that the up-projection costs no exposed load latency.
    constexpr int NBQ = HEAVY ? 8 : 4;               // 8-element chunks of a row of B held per lane
    const bool fast_fin = (p.rank > 0) && (p.rank <= 16 * NBQ) && (p.SK == 1);
    uint4 bq[NBQ];
    auto b_prefetch = [&](int tile) {
        const int row = lane >> 1, n = tile * kTileRows + row;
        const T *own = own_b(tile);
        const T *src = own ? own + (size_t)row * p.rank : static_cast<const T *>(p.B) + (size_t)n * p.rank;
#pragma unroll
        for (int i = 0; i < NBQ; ++i) {
            const int c = (lane & 1) + 2 * i;
            bq[i] = make_uint4(0u, 0u, 0u, 0u);
            if (8 * c < p.rank && n < p.N)
                bq[i] = own ? *reinterpret_cast<const uint4 *>(src + 8 * c) : __ldg(reinterpret_cast<const uint4 *>(src + 8 * c));
        }
    };
    // y rows of `tile` = staged main sums + t.B^T from the prefetched chunks
    auto finish_fast = [&](int tile) {
        const int row = lane >> 1, n = tile * kTileRows + row;
#pragma unroll 1
        for (int m = 0; m < p.M; ++m) {
            float sub = 0.f;
#pragma unroll
            for (int i = 0; i < NBQ; ++i) {
                const int c = (lane & 1) + 2 * i;
                if (8 * c < p.rank) {
                    const float4 t0 = *reinterpret_cast<const float4 *>(s_t + (size_t)m * p.rank + 8 * c);
                    const float4 t1 = *reinterpret_cast<const float4 *>(s_t + (size_t)m * p.rank + 8 * c + 4);
                    const float2 b0 = Pk<T>::to_float2(bq[i].x), b1 = Pk<T>::to_float2(bq[i].y);
                    const float2 b2 = Pk<T>::to_float2(bq[i].z), b3 = Pk<T>::to_float2(bq[i].w);
                    sub = fmaf(t0.x, b0.x, sub); sub = fmaf(t0.y, b0.y, sub);
                    sub = fmaf(t0.z, b1.x, sub); sub = fmaf(t0.w, b1.y, sub);
                    sub = fmaf(t1.x, b2.x, sub); sub = fmaf(t1.y, b2.y, sub);
                    sub = fmaf(t1.z, b3.x, sub); sub = fmaf(t1.w, b3.y, sub);
                }
            }
            sub += __shfl_xor_sync(0xffffffffu, sub, 1);
            if ((lane & 1) == 0 && n < p.N)
                static_cast<T *>(p.y)[(size_t)m * p.N + n] = ActTraits<T>::from_float(s_stage[m * kTileRows + row] + sub);
        }
        ++n_retired;
    };
    // Up-projection of all rows of this CTA at once (light variant, one K slice, B of the own tiles in
    // shared memory, M <= 4, rank a multiple of 16): once t is complete it becomes eight 16-bit columns
    // (tokens 0..3 rounded, then the remainders of that rounding), and per tile rank / 16 MMAs
    // (rows of B x columns of t) give t.B^T for its 16 rows.  A tile is then finished by adding
    // two numbers per output.  Tiles that are done before t is wait in their segment buffers for
    // as long as that holds nobody up.
    T *s_th = reinterpret_cast<T *>(s_stage + kTileRows * kDecodeMaxM);       // [8 columns][rank]
    const bool sub_at_once = !HEAVY && fast_fin && b_in_smem && p.M <= 4 && (p.rank % 16) == 0 && !p.t_late;
    bool sub_done = false;          // t is there as 16-bit columns
    float isc = 1.f;
    auto make_sub = [&]() {
        // fp16 columns: a power of two keeps a large t inside the format (exact, undone in the finish)
        float sc = 1.f;
        if (std::is_same<T, __half>::value) {
            float tmax = 0.f;
            for (int i = lane; i < p.M * p.rank; i += 32) tmax = fmaxf(tmax, fabsf(s_t[i]));
            for (int o = 16; o > 0; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
            if (tmax >= 16384.f) {
                int e = 0;
                (void)frexpf(tmax, &e);
                sc = ldexpf(1.f, 14 - e);
                isc = ldexpf(1.f, e - 14);
            }
        }
        for (int j = lane; j < p.rank; j += 32)
#pragma unroll
            for (int m = 0; m < 4; ++m) {
                float hi = 0.f, lo = 0.f;
                if (m < p.M) {
                    const float tv = s_t[m * p.rank + j] * sc;
                    hi = tv;
                    lo = tv - ActTraits<T>::to_float(ActTraits<T>::from_float(tv));
                }
                s_th[m * p.rank + j] = ActTraits<T>::from_float(hi);
                s_th[(4 + m) * p.rank + j] = ActTraits<T>::from_float(lo);
            }
        __syncwarp();
        sub_done = true;
    };
    // One tile: t.B^T of its 16 rows by rank / 16 MMAs (the result has the layout of the main sums: lane
    // (g, tq < 2) holds tokens 2 tq, 2 tq + 1 of rows g and g + 8), added to the main sums in registers,
    // rounded and stored.
    auto finish_sub = [&](int tile, int seg, const float (&main)[4]) {
        const uint32_t *tcol = reinterpret_cast<const uint32_t *>(s_th + (size_t)g * p.rank);
        const uint32_t *ba = reinterpret_cast<const uint32_t *>(s_B + (size_t)(seg * kTileRows + g) * p.rank);
        const uint32_t *bb = ba + 4 * p.rank;                                // row g + 8
        float d[4] = {0.f, 0.f, 0.f, 0.f};
        const int nk16 = p.rank / 16;                                        // at most 4 here (rank <= 64): all loads go out first
        uint32_t a[4][4], tb[4][2];
#pragma unroll
        for (int k16 = 0; k16 < 4; ++k16) {
            const int w = k16 * 8 + tq;
            const bool on = k16 < nk16;
            a[k16][0] = on ? ba[w] : 0u;
            a[k16][1] = on ? bb[w] : 0u;
            a[k16][2] = on ? ba[w + 4] : 0u;
            a[k16][3] = on ? bb[w + 4] : 0u;
            tb[k16][0] = on ? tcol[w] : 0u;
            tb[k16][1] = on ? tcol[w + 4] : 0u;
        }
#pragma unroll
        for (int k16 = 0; k16 < 4; ++k16) Pk<T>::mma(d, a[k16], tb[k16][0], tb[k16][1]);
#pragma unroll
        for (int q = 0; q < 4; ++q) d[q] = (d[q] + __shfl_xor_sync(0xffffffffu, d[q], 2)) * isc;   // rounded part + remainder
        if (tq < p.vt) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int n = tile * kTileRows + g + 8 * (i >> 1), m = 2 * tq + (i & 1);
                if (m < p.M && n < p.N) static_cast<T *>(p.y)[(size_t)m * p.N + n] = ActTraits<T>::from_float(main[i] + d[i]);
            }
        }
        ++n_retired;
    };
    // Waits for t while that costs nothing: until it is complete, or the compute warps are about to
    // run out of segment buffers, or they are through with all segments (then the tile is parked as
    // before: a CTA never holds its SM just to wait for other CTAs).
    auto wait_t_with_slack = [&](int seg) {
        const int last = min(seg + p.nbuf, nseg - 1);
        if (last <= seg) return;
        const uint32_t bar = seg_full + 8u * (uint32_t)(last % p.nbuf), par = (uint32_t)(last / p.nbuf) & 1u;
#pragma unroll 1
        for (uint32_t i = 0; i < kWaitLimit; ++i) {
            if (t_poll()) return;
            if (mbar_test(bar, par)) return;
            __nanosleep(200);
        }
    };
    // Finish `tile` from scratch slots (all contributions are there and visible).
    auto finish_from_slots = [&](int tile) {
        finish_tile<T>(static_cast<T *>(p.y), p.partial + (size_t)tile * p.maxslots * p.M * kTileRows,
                       static_cast<const T *>(p.B), p.M, p.N, p.rank, tile, lane, nullptr, 0, p.SK, s_t, own_b(tile));
        ++n_retired;
        if (p.rank == 0 && lane == 0) p.ctr[kCtrFirstTile + tile] = 0;   // nobody else will touch it again
    };
    // Copies the staged sums of this warp to its scratch slot of `tile`.
    auto stage_to_slot = [&](int tile) {
        float *slot = p.partial + ((size_t)tile * p.maxslots + s) * p.M * kTileRows;
        for (int idx = lane; idx < kTileRows * p.M; idx += 32) slot[idx] = s_stage[idx];
        __syncwarp();
    };

    // After this CTA's share of t is in: count it; the warp that completes t publishes
    // the flag and finishes every tile that was parked (by any CTA) before the flag was up.
    auto t_arrive = [&]() {
        __syncwarp();
        int done = 0;
        if (lane == 0) {
            __threadfence();
            done = (atomicAdd(p.ctr + kCtrT, 1) == p.t_target - 1);
        }
        done = __shfl_sync(0xffffffffu, done, 0);
        if (!done) return;
        int npend = 0;
        if (lane == 0) {
            p.ctr[kCtrT] = 0;
            __threadfence();
            atomicExch(p.ctr + kCtrReady, 1);
            __threadfence();
            npend = ld_acquire(p.ctr + kCtrPendingN);
        }
        npend = __shfl_sync(0xffffffffu, npend, 0);
        (void)t_poll();
#pragma unroll 1
        for (int i = 0; i < npend; ++i) {
            int tile = 0;
            if (lane == 0) tile = ld_acquire(p.ctr + kCtrFirstTile + p.NT + i) - 1;
            tile = __shfl_sync(0xffffffffu, tile, 0);
            if (tile < 0) continue;                    // entry not visible yet: its owner will see the flag
            if (!tile_claim(p, tile, lane)) continue;
            __threadfence();
            finish_from_slots(tile);
        }
        ++n_retired;                                   // the completer's own token in the retire count
    };

    if (has_t && !p.t_late) {
        if (t_by_compute) {
            if (!mbar_wait(t_done, 0)) dead = true;     // the compute warps' units are in
        } else if (!t_units_mma()) {
            dead = true;
        }
        trace_mark(p, 3);
    }
    if (!HEAVY && p.ab_alias && b_in_smem) {
        // A and the staged x are used up: their place goes to B of the own tiles (needed once t is complete)
        __syncwarp();
        if (lane == 0) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            const uint32_t bytes = (uint32_t)b_rows * p.rank * 2u;
            mbar_expect_tx(b_full, bytes);
            bulk_g2s(smem_u32(s_B), static_cast<const T *>(p.B) + (size_t)tile_first * kTileRows * p.rank, bytes, b_full);
        }
    }
    if (has_t && !p.t_late) t_arrive();
    trace_mark(p, 4);
    if (b_in_smem && !mbar_wait(b_full, 0)) dead = true;

    long long e_wait = 0, e_sum = 0, e_fin = 0;      // trace: cycles waiting for segments, adding partials, finishing (fast path)
#pragma unroll 1
    for (int seg = 0; seg < nseg && !dead; ++seg) {
        const int buf = seg % p.nbuf;
        const int tile = tile_first + seg;
        const int cnt = p.SK, myslot = s;       // one contribution per K slice
        // While the compute warps still work on the segment, look whether every other
        // contribution of a shared tile has already arrived.
        int others_in = 0;
        if (cnt > 1) {
            if (lane == 0) others_in = ((ld_acquire(p.ctr + kCtrFirstTile + tile) & 0xFFFF) == cnt - 1);
            others_in = __shfl_sync(0xffffffffu, others_in, 0);
        }
        if (fast_fin && !sub_at_once) b_prefetch(tile);
        const long long c_w0 = p.trace ? clock64() : 0;
        if (!mbar_wait_idle(seg_full + 8u * buf, (uint32_t)(seg / p.nbuf) & 1u)) {
            dead = true;
            break;
        }
        const long long c_w1 = p.trace ? clock64() : 0;
        e_wait += c_w1 - c_w0;
        trace_mark(p, seg == 0 ? 5 : 7);
        // add the eight warps' partial tiles in warp order and stage the result as [token][row]
        float acc[MT][4];
#pragma unroll
        for (int b = 0; b < MT; ++b) acc[b][0] = acc[b][1] = acc[b][2] = acc[b][3] = 0.f;
        if (tq < p.vt) {
            const float4 *src = reinterpret_cast<const float4 *>(s_seg + (size_t)buf * segbuf_floats);
#pragma unroll
            for (int w = 0; w < kCW; ++w)
#pragma unroll
                for (int b = 0; b < MT; ++b) {
                    const float4 v = src[(size_t)((w * 8 + g) * p.vt + tq) * MT + b];
                    acc[b][0] += v.x; acc[b][1] += v.y; acc[b][2] += v.z; acc[b][3] += v.w;
                }
#pragma unroll
            for (int b = 0; b < MT; ++b)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int row = g + 8 * (i >> 1), m = 8 * b + 2 * tq + (i & 1);
                    if (m < p.M) s_stage[m * kTileRows + row] = acc[b][i];
                }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(seg_free + 8u * buf);
        const long long c_w2 = p.trace ? clock64() : 0;
        e_sum += c_w2 - c_w1;

        if (cnt == 1 || others_in) {
            // This warp finishes the tile: straight from the staged sums if t is complete ...
            if (sub_at_once && p.t_wait && !t_local) wait_t_with_slack(seg);
            if (p.n_t > 0 && !t_local) {
                // t comes from the CTAs at the head of this grid, which wait for nothing: wait for it (bounded)
                bool ok = false;
#pragma unroll 1
                for (uint32_t i = 0; i < kWaitLimit && !ok; ++i) {
                    ok = t_poll();
                    if (!ok) __nanosleep(200);
                }
                if (!ok) {
                    dead = true;
                    break;
                }
            }
            if (t_poll()) {
                if (sub_at_once) {
                    if (!sub_done) {
                        trace_mark(p, 3);
                        make_sub();
                        trace_mark(p, 14);
                    }
                    finish_sub(tile, seg, acc[0]);
                    __syncwarp();
                    if (p.trace) e_fin += clock64() - c_w2;
                    continue;
                }
                if (fast_fin) {
                    finish_fast(tile);
                    __syncwarp();
                    if (p.trace) e_fin += clock64() - c_w2;
                    continue;
                }
                finish_tile<T>(static_cast<T *>(p.y), p.partial + (size_t)tile * p.maxslots * p.M * kTileRows,
                               static_cast<const T *>(p.B), p.M, p.N, p.rank, tile, lane, s_stage, myslot, cnt, s_t,
                               own_b(tile));
                ++n_retired;
                if (p.rank == 0 && cnt > 1 && lane == 0) p.ctr[kCtrFirstTile + tile] = 0;
                __syncwarp();
                continue;
            }
            // ... else its sums wait in scratch on a local list until t is.
            stage_to_slot(tile);
            if (lane == 0) s_def[n_def] = tile;
            ++n_def;
            __syncwarp();
            continue;
        }
        // Shared tile, others still missing: leave the partial and an arrival count.
        stage_to_slot(tile);
        int last = 0;
        if (lane == 0) {
            __threadfence();
            last = ((atomicAdd(p.ctr + kCtrFirstTile + tile, 1) & 0xFFFF) == cnt - 1);
        }
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
            if (lane == 0) s_def[n_def] = tile;
            ++n_def;
            __syncwarp();
        }
    }
    trace_mark(p, 8);

    if (has_t && p.t_late) {
        if (!t_units(tu0, 1)) dead = true;
        t_arrive();
    }
    // ---- tiles this warp still owes: finish them once t is complete, else park them
    // globally for the warp that completes t ----
    if (n_def > 0) {
        __threadfence();
        // t is normally complete within a microsecond or two of the first tiles: look a bounded
        // number of times before handing the tiles over (every CTA contributes to t before it
        // waits for anything, so this cannot block the contributors)
        bool ready = false;
#pragma unroll 1
        for (int spin = 0; spin <= kTPolls && !ready; ++spin) ready = t_poll();
        if (p.n_t > 0 && !ready) {
            // t comes from the CTAs at the head of the grid, and nobody would pick parked tiles up: wait (bounded)
#pragma unroll 1
            for (uint32_t i = 0; i < kWaitLimit && !ready; ++i) {
                ready = t_poll();
                if (!ready) __nanosleep(200);
            }
            if (!ready) {
                dead = true;
                n_def = 0;
            }
        }
#pragma unroll 1
        for (int i = 0; i < n_def; ++i) {
            const int tile = s_def[i];
            if (!ready) {
                int st = 0;
                if (lane == 0) {
                    // park the tile, then look again: either we see the flag now, or the warp
                    // that raises it will see our entry (both sides fence in between)
                    const int idx = atomicAdd(p.ctr + kCtrPendingN, 1);
                    atomicExch(p.ctr + kCtrFirstTile + p.NT + idx, tile + 1);
                    __threadfence();
                    st = ld_acquire(p.ctr + kCtrReady);
                }
                st = __shfl_sync(0xffffffffu, st, 0);
                if (!st || !tile_claim(p, tile, lane)) continue;     // parked (or already taken)
                __threadfence();
                ready = t_poll();
            }
            finish_from_slots(tile);
        }
    }
    if (dead && lane == 0) atomicExch(p.status, (int)FBQ_ERR_TIMEOUT);

    // ---- retire: whoever brings the count to NT + 1 (every tile finished, and the t-completing
    // warp out of its parked-tile loop) restores the scratch invariants for the next call ----
    if (p.rank > 0 && n_retired > 0) {
        __syncwarp();
        int fin = 0;
        if (lane == 0) {
            __threadfence();
            fin = (atomicAdd(p.ctr + kCtrDone, n_retired) + n_retired == p.NT + 1);
        }
        fin = __shfl_sync(0xffffffffu, fin, 0);
        if (fin) {
            __threadfence();
            for (int i = lane; i < 2 * p.NT; i += 32) p.ctr[kCtrFirstTile + i] = 0;   // arrivals + parked list
            for (int i = lane; i < p.M * p.rank; i += 32) p.t[i] = 0.f;
            if (lane == 0) {
                p.ctr[kCtrDone] = 0;
                p.ctr[kCtrReady] = 0;
                p.ctr[kCtrPendingN] = 0;
            }
        }
    }
    trace_mark(p, 9);
    if (p.trace && lane == 0) {
        unsigned long long *row = p.trace + ((size_t)blockIdx.x * kWarps + warp) * 16;
        row[10] = (unsigned long long)e_wait;
        row[11] = (unsigned long long)e_sum;
        row[12] = (unsigned long long)e_fin;
        row[13] = (unsigned long long)n_def;
    }
}

template <int BITS, typename T, int MT, bool HEAVY, bool I8>
__global__ void __launch_bounds__(kThreads, 2) decode_kernel(const __grid_constant__ DecodeParams p,
                                                             const __grid_constant__ CUtensorMap wmap)
{
    decode_body<BITS, T, MT, HEAVY, I8>(p, &wmap, (int)blockIdx.x);
}

// Several independent problems in one grid: CTAs first[i] .. first[i+1]-1 run problem i exactly as
// a launch of its own would (its own scratch, counters and shared-memory plan); the CTAs of all
// problems are resident together and nothing synchronises across problems.
constexpr int kBatchMax = 8;
struct DecodeBatch {
    CUtensorMap wmap[kBatchMax];
    DecodeParams prob[kBatchMax];
    int first[kBatchMax + 1];
    int count;
};
template <int BITS, typename T, int MT, bool HEAVY, bool I8>
__global__ void __launch_bounds__(kThreads, 2) decode_batch_kernel(const __grid_constant__ DecodeBatch b)
{
    int pi = 0;
    while (pi + 1 < b.count && (int)blockIdx.x >= b.first[pi + 1]) ++pi;
    decode_body<BITS, T, MT, HEAVY, I8>(b.prob[pi], &b.wmap[pi], (int)blockIdx.x - b.first[pi]);
}

// ------------------------------------------------------------------ host side
struct Plan {
    int SK, R, NT, CHG, NS, nbuf, t_target, maxslots, vt, a_cap, b_cap_rows, meta_rows;
    int x_pitch, stage_bytes;
    int off_tab, off_def, off_meta, off_x, off_px, off_segbuf, off_A, off_B, off_t, off_ring;
    size_t smem;
    bool ok;
    bool i8;            // codes and x go to the tensor cores as 8-bit integers (M <= 2)
    bool heavy;         // the compute warps take the units of the down-projection
    int ab_alias;
    int n_t;            // CTAs at the head of the grid that compute t (0: every CTA contributes)
};

int g_sm_count = 0;
int g_t_late = 0, g_t_wait = 1;
constexpr size_t kSmemBudget = 112 * 1024;   // two CTAs (this launch and the next one) fit on an SM (228 KB, 1 KB reserved per CTA)
constexpr size_t kSmemMax = 227 * 1024;      // everything an SM has

Plan make_plan(const LinearArgs &a, const DecodeTuning &tune)
{
    Plan pl{};
    pl.ok = false;
    if (g_sm_count == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return pl;
        if (cudaDeviceGetAttribute(&g_sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return pl;
    }
    const int GB = (a.bits == 4) ? 64 : 48;
    const int G = a.K / kGroupFast;
    const int mt = (a.M <= 8) ? 1 : 2;
    pl.NT = (a.N + kTileRows - 1) / kTileRows;
    int max_ctas = 2 * g_sm_count;            // two CTAs per SM: one streams while the other starts or ends
    if (tune.max_ctas > 0) max_ctas = min(max_ctas, tune.max_ctas);
    pl.vt = (mt == 2) ? 4 : min(4, (a.M + 1) / 2);
    pl.i8 = tune.i8 != 0 && a.M <= kI8MaxM;
    // K slices: one, unless the x slice and the other tables do not fit next to the ring.
    // First try to stay within half an SM's shared memory (so that this launch and the next
    // one can be resident together) with few slices; otherwise take the whole SM.
    auto layout = [&](int sk, size_t budget, bool many_buffers, int chg_cap) {
        pl.SK = sk;
        const int ngs_max = (G + sk - 1) / sk;
        pl.R = max(1, min(max_ctas / sk, pl.NT));
        const int nseg_max = (pl.NT + pl.R - 1) / pl.R;
        pl.maxslots = sk;
        pl.CHG = max(1, min(min(tune.chunk > 0 ? tune.chunk : 16, chg_cap), ngs_max));
        pl.stage_bytes = kTileRows * pl.CHG * GB;             // [group][row][GB], dense
        pl.x_pitch = ngs_max * kGroupFast + 32;    // +64 bytes: tokens 2j, 2j+1 land in different bank halves
        const int nkc = (ngs_max * kGroupFast + kTUnitK - 1) / kTUnitK;
        long long tu_max = 0;                                 // most units any CTA gets
        for (int r = 0; r < pl.R && r < 2 * nkc + 2; ++r) {   // the ranges repeat with period nkc; the first CTAs have the largest
            int u0, u1;
            unit_range(r, pl.R, a.rank, nkc, &u0, &u1);
            tu_max = max(tu_max, (long long)(u1 - u0));
        }
        if (pl.R < nkc) tu_max = ((long long)a.rank * nkc + pl.R - 1) / pl.R;
        pl.a_cap = (int)min(tu_max, 8LL);
        // Heavy sub-branch: rank above what the light tile finish holds, or more units of the down-projection
        // per CTA than its epilogue warp should take by itself (tensor-core form: what fits its staging
        // area; plain form: (token, unit) pairs).
        // t from a few CTAs at the head of the grid (M <= 4; over all of K, whatever the K slices): then the others hold no A
        pl.n_t = 0;
        if (a.rank > 0 && a.M <= kTMmaMaxM && !g_t_late && tune.t_ctas != 0) {
            const int nblocks = ((a.K + kTcK - 1) / kTcK) * ((a.rank + 7) / 8);            // over all of K
            pl.n_t = min(12, (nblocks + kTWarps - 1) / kTWarps);
            pl.a_cap = 0;
            tu_max = 0;
        }
        pl.heavy = a.rank > 64 || (a.rank > 0 && (a.M <= kTMmaMaxM ? tu_max > 8 : tu_max * a.M > kTUnitsOneWarp));
        pl.ab_alias = (a.rank > 0 && !pl.heavy && !g_t_late && pl.n_t == 0) ? 1 : 0;
        size_t off = (size_t)(2 * 8 + 2 * kNBufMax + 4) * 8;      // room for up to 8 stages' barriers
        off = (off + 15) & ~(size_t)15;
        pl.off_tab = (int)off;
        pl.off_def = (int)off;
        off += (size_t)(kMaxSeg + 2) * sizeof(int);
        off = (off + 15) & ~(size_t)15;
        pl.off_meta = (int)off;
        pl.meta_rows = nseg_max * kTileRows;
        off += (size_t)pl.meta_rows * (ngs_max | 1) * 8;
        off = (off + 127) & ~(size_t)127;
        pl.off_x = (int)off;
        // x of the slice: 16-bit values per token, or (integer form) three one-byte columns per value, 36 slots per 32 values
        off += pl.i8 ? (size_t)ngs_max * (3 * a.M) * 144 : (size_t)a.M * pl.x_pitch * 2;
        off = (off + 127) & ~(size_t)127;
        pl.off_px = (int)off;
        off += (size_t)ngs_max * 8 * mt * 8;
        off = (off + 127) & ~(size_t)127;
        pl.off_segbuf = (int)off;
        pl.nbuf = (many_buffers && (size_t)kCW * 8 * pl.vt * 4 * mt * 4 <= 1024) ? kNBufMax : 4;   // small tiles (M <= 2): more of them may wait for t
        off += (size_t)pl.nbuf * kCW * 8 * pl.vt * 4 * mt * 4;
        off = (off + 127) & ~(size_t)127;
        pl.off_A = (int)off;
        const size_t b_bytes = (size_t)nseg_max * kTileRows * a.rank * 2;
        const size_t a_bytes = pl.n_t > 0 ? 0 : (size_t)(pl.a_cap + (a.rank > 0 && a.M <= kTMmaMaxM ? a.M : 0)) * kAPitch * 2;   // units of A, then x of one k chunk
        off += pl.ab_alias ? max(a_bytes, b_bytes) : a_bytes;
        off = (off + 127) & ~(size_t)127;
        pl.off_t = (int)off;
        off += (size_t)a.M * a.rank * 4 + (size_t)kTileRows * kDecodeMaxM * 4;   // t, then the epilogue warp's staging tile
        off += (size_t)8 * a.rank * 2;                                            // t as 16-bit columns
        off = (off + 127) & ~(size_t)127;
        // what is left: two stages of the ring, then B of the own tiles, then more stages
        pl.off_B = (int)off;
        int ns_want = tune.depth > 0 ? tune.depth : 4;
        ns_want = max(2, min(ns_want, 8));
        pl.b_cap_rows = 0;
        if (pl.ab_alias) {
            pl.off_B = pl.off_A;
            pl.b_cap_rows = nseg_max * kTileRows;
        } else if (off + b_bytes + (size_t)2 * pl.stage_bytes <= budget) {      // B of the own tiles before a third and fourth stage
            pl.b_cap_rows = nseg_max * kTileRows;
            off += b_bytes;
            off = (off + 127) & ~(size_t)127;
        }
        pl.off_ring = (int)off;
        pl.NS = ns_want;
        while (pl.NS > 2 && off + (size_t)pl.NS * pl.stage_bytes > budget) --pl.NS;
        off += (size_t)pl.NS * pl.stage_bytes;
        if (pl.n_t > 0) off = max(off, (size_t)1024 + (size_t)kTWarps * (8 + a.M) * kTcPitch * 2);  // what a t CTA needs
        pl.smem = off;
        return nseg_max <= kMaxSeg && pl.smem <= budget;
    };
    // the integer form first; where its larger x does not fit, the 16-bit form before more K slices
    const bool want_i8 = pl.i8;
    auto either = [&](int sk, size_t budget) {
        for (int form = 0; form < (want_i8 ? 2 : 1); ++form) {
            pl.i8 = want_i8 && form == 0;
            // stages of 16 groups, else of 8 (more hand-overs per byte, but still one K slice)
            // B of the own tiles in shared memory (tensor-core tile finish) is worth more than eight segment
            // buffers: a layout without it is taken only if none with it fits
            for (int chg = 16; chg >= 8; chg -= 8) {
                const bool with_many = layout(sk, budget, true, chg);
                if (with_many && (a.rank == 0 || pl.b_cap_rows > 0)) return true;
                if (layout(sk, budget, false, chg) && (a.rank == 0 || pl.b_cap_rows > 0)) return true;
                if (with_many) return layout(sk, budget, true, chg);
                if (layout(sk, budget, false, chg)) return true;
            }
        }
        return false;
    };
    if (tune.sk > 0) {
        pl.ok = either(min(tune.sk, G), kSmemMax);
    } else {
        for (int sk = 1; sk <= min(G, 4) && !pl.ok; ++sk) pl.ok = either(sk, kSmemBudget);
        for (int sk = 1; sk <= G && !pl.ok; ++sk) pl.ok = either(sk, kSmemMax);
    }
    if (getenv("FBQ_PLAN"))
        fprintf(stderr, "plan M %d N %d K %d r %d: ok %d SK %d R %d CHG %d NS %d nbuf %d a_cap %d b_rows %d smem %zu (meta %d x %d ring@%d) i8 %d heavy %d alias %d n_t %d\n", a.M, a.N, a.K,
                a.rank, (int)pl.ok, pl.SK, pl.R, pl.CHG, pl.NS, pl.nbuf, pl.a_cap, pl.b_cap_rows, pl.smem, pl.off_x - pl.off_meta,
                pl.off_px - pl.off_x, pl.off_ring, (int)pl.i8, (int)pl.heavy, pl.ab_alias, pl.n_t);
    // CTAs that own at least one unit of the down-projection
    pl.t_target = 0;
    if (pl.n_t > 0) {
        pl.t_target = pl.n_t;
    } else if (a.rank > 0) {
        for (int s = 0; s < pl.SK; ++s) {
            const int ngs = (int)((long long)(s + 1) * G / pl.SK) - (int)((long long)s * G / pl.SK);
            const int nkc = (ngs * kGroupFast + kTUnitK - 1) / kTUnitK;
            for (int r = 0; r < pl.R; ++r) {
                int u0, u1;
                unit_range(r, pl.R, a.rank, nkc, &u0, &u1);
                pl.t_target += (u1 > u0) ? 1 : 0;
            }
        }
    }
    return pl;
}

// 3-D tensor map of the packed codes for the weight stream: (word in group, weight row, group), boxes of
// one group's words x 16 rows x CHG groups, which land in shared memory as [group][row][GB bytes].
// Encoding takes a microsecond or two on the host, so the last maps are kept (they depend on the
// weights' address and the plan only).
struct MapKey {
    const void *qw;
    int N, G, bits, chg;
    bool operator==(const MapKey &o) const { return qw == o.qw && N == o.N && G == o.G && bits == o.bits && chg == o.chg; }
};
cudaError_t weight_map(CUtensorMap *map, const LinearArgs &a, const Plan &pl)
{
    static std::mutex mu;
    static std::vector<std::pair<MapKey, CUtensorMap>> cache;
    static size_t next = 0;
    static PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
    const MapKey key{a.qw, a.N, a.K / kGroupFast, a.bits, pl.CHG};
    std::lock_guard<std::mutex> lk(mu);
    for (const auto &e : cache)
        if (e.first == key) {
            *map = e.second;
            return cudaSuccess;
        }
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess) return e;
        if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
        encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
    }
    const cuuint32_t wpg = (a.bits == 4) ? 16 : 12;
    const cuuint64_t dims[3] = {wpg, (cuuint64_t)a.N, (cuuint64_t)key.G};
    const cuuint64_t strides[2] = {(cuuint64_t)key.G * wpg * 4, (cuuint64_t)wpg * 4};
    const cuuint32_t box[3] = {wpg, (cuuint32_t)kTileRows, (cuuint32_t)pl.CHG};
    const cuuint32_t estr[3] = {1, 1, 1};
    if (encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<uint32_t *>(a.qw), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    constexpr size_t kKeep = 256;
    if (cache.size() < kKeep)
        cache.emplace_back(key, *map);
    else
        cache[next++ % kKeep] = std::make_pair(key, *map);
    return cudaSuccess;
}

template <int BITS, typename T, int MT, bool HEAVY, bool I8>
cudaError_t launch_variant(const DecodeParams &p, const CUtensorMap &wmap, const Plan &pl, bool pdl, cudaStream_t s)
{
    auto kern = decode_kernel<BITS, T, MT, HEAVY, I8>;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemMax);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(pl.n_t + pl.R * pl.SK));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, p, wmap);
}

}  // namespace

void decode_set_test_switch(int t_late) { g_t_late = t_late; }
void decode_set_t_wait(int on) { g_t_wait = on; }

void decode_workspace_need(const LinearArgs &a, const DecodeTuning &tune, size_t *partial_floats, int *counters)
{
    const Plan pl = make_plan(a, tune);
    *partial_floats = (size_t)pl.NT * pl.maxslots * a.M * kTileRows;
    *counters = kCtrFirstTile + 2 * pl.NT;
}

namespace {
template <typename X> struct TypeTag { using type = X; };

// Calls f(bits, activation type, MT, HEAVY, I8) with compile-time tags for this problem (the integer
// form exists for one token block only).
template <typename F>
cudaError_t dispatch_variant(const LinearArgs &a, F f, bool heavy, bool i8)
{
    auto with_heavy = [&](auto bits, auto type, auto mt, auto e4) {
        return heavy ? f(bits, type, mt, std::true_type{}, e4) : f(bits, type, mt, std::false_type{}, e4);
    };
    auto with_mt = [&](auto bits, auto type) {
        if (i8) return with_heavy(bits, type, std::integral_constant<int, 1>{}, std::true_type{});
        return (a.M <= 8) ? with_heavy(bits, type, std::integral_constant<int, 1>{}, std::false_type{})
                          : with_heavy(bits, type, std::integral_constant<int, 2>{}, std::false_type{});
    };
    auto with_type = [&](auto bits) { return a.bf16 ? with_mt(bits, TypeTag<__nv_bfloat16>{}) : with_mt(bits, TypeTag<__half>{}); };
    return (a.bits == 4) ? with_type(std::integral_constant<int, 4>{}) : with_type(std::integral_constant<int, 3>{});
}

DecodeParams fill_params(const LinearArgs &a, const Plan &pl, float *partial, float *t, int *ctr, int *status, void *trace)
{
    DecodeParams p{};
    p.x = a.x;
    p.qw = reinterpret_cast<const uint8_t *>(a.qw);
    p.scales = a.scales;
    p.zeros = a.zeros;
    p.A = a.A;
    p.B = a.B;
    p.y = a.y;
    p.partial = partial;
    p.t = t;
    p.ctr = ctr;
    p.status = status;
    p.M = a.M; p.N = a.N; p.K = a.K; p.G = a.K / kGroupFast; p.rank = a.rank;
    p.SK = pl.SK; p.R = pl.R; p.NT = pl.NT; p.CHG = pl.CHG; p.NS = pl.NS; p.nbuf = pl.nbuf;
    p.maxslots = pl.maxslots;
    p.t_target = pl.t_target;
    p.n_t = pl.n_t;
    p.t_late = g_t_late;
    p.vt = pl.vt;
    p.x_pitch = pl.x_pitch; p.stage_bytes = pl.stage_bytes;
    p.a_cap = pl.a_cap; p.b_cap_rows = pl.b_cap_rows; p.ab_alias = pl.ab_alias; p.t_wait = g_t_wait;
    p.meta_rows = pl.meta_rows;
    p.off_tab = pl.off_tab; p.off_def = pl.off_def; p.off_meta = pl.off_meta; p.off_x = pl.off_x; p.off_px = pl.off_px;
    p.off_segbuf = pl.off_segbuf; p.off_A = pl.off_A; p.off_B = pl.off_B; p.off_t = pl.off_t; p.off_ring = pl.off_ring;
    p.trace = reinterpret_cast<unsigned long long *>(trace);
    return p;
}

template <int BITS, typename T, int MT, bool HEAVY, bool I8>
cudaError_t launch_batch_variant(const DecodeBatch &b, size_t smem, bool pdl, cudaStream_t s)
{
    auto kern = decode_batch_kernel<BITS, T, MT, HEAVY, I8>;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemMax);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)b.first[b.count]);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, b);
}
}  // namespace

cudaError_t launch_decode(const LinearArgs &a, Workspace &ws, const DecodeTuning &tune, cudaStream_t s, int *launches)
{
    const Plan pl = make_plan(a, tune);
    if (!pl.ok) return cudaErrorInvalidConfiguration;
    const DecodeParams p = fill_params(a, pl, ws.partial, ws.t, ws.counters, ws.counters + kCtrStatus, ws.trace);
    CUtensorMap wmap;
    if (cudaError_t me = weight_map(&wmap, a, pl); me != cudaSuccess) return me;
    const bool pdl = tune.pdl != 0;
    const bool heavy = pl.heavy;
    cudaError_t e = dispatch_variant(a, [&](auto bits, auto type, auto mt, auto hv, auto e4) {
        return launch_variant<decltype(bits)::value, typename decltype(type)::type, decltype(mt)::value, decltype(hv)::value,
                              decltype(e4)::value>(p, wmap, pl, pdl, s);
    }, heavy, pl.i8);
    if (e == cudaSuccess) ++*launches;
    return e;
}

// ---- several problems in one launch ---------------------------------------------------------
int decode_batch_max() { return kBatchMax; }

// Scratch the batch needs in one workspace: partial floats, t floats and counters, summed over the
// problems (problem i is planned with at most ctas[i] CTAs).  false if a problem has no plan.
bool decode_batch_need(const LinearArgs *a, int count, const int *ctas, const DecodeTuning &tune, size_t *partial_floats,
                       size_t *t_floats, int *counters)
{
    *partial_floats = 0;
    *t_floats = 0;
    *counters = kCtrFirstTile;                      // the shared head (status word) comes first
    bool i8 = false, heavy = false;
    for (int i = 0; i < count; ++i) {
        DecodeTuning tn = tune;
        tn.max_ctas = ctas[i];
        const Plan pl = make_plan(a[i], tn);
        if (!pl.ok) return false;
        // One launch runs ONE kernel variant: every problem's shared-memory layout must have been planned for
        // the same form (integer or 16-bit) and the same sub-branch variant.  Plans that disagree (the form
        // falls back where x of a long K does not fit) go to one launch per problem instead.
        if (i == 0) {
            i8 = pl.i8;
            heavy = pl.heavy;
        } else if (pl.i8 != i8 || pl.heavy != heavy) {
            return false;
        }
        *partial_floats += (size_t)pl.NT * pl.maxslots * a[i].M * kTileRows;
        *t_floats += (size_t)kDecodeMaxM * kMaxRank;
        *counters += kCtrFirstTile + 2 * pl.NT;
    }
    return true;
}

// All problems share M, bits, rank and the activation type.  ws must hold decode_batch_need().
cudaError_t launch_decode_batch(const LinearArgs *a, int count, const int *ctas, Workspace &ws, const DecodeTuning &tune,
                                cudaStream_t s, int *launches)
{
    if (count < 1 || count > kBatchMax) return cudaErrorInvalidConfiguration;
    DecodeBatch b{};
    b.count = count;
    size_t smem = 0, off_p = 0, off_t = 0;
    int off_c = kCtrFirstTile;
    bool heavy = false, i8 = false;
    for (int i = 0; i < count; ++i) {
        DecodeTuning tn = tune;
        tn.max_ctas = ctas[i];
        const Plan pl = make_plan(a[i], tn);
        if (!pl.ok) return cudaErrorInvalidConfiguration;
        i8 = pl.i8;                                   // the same for all problems: they share M
        if (cudaError_t me = weight_map(&b.wmap[i], a[i], pl); me != cudaSuccess) return me;
        b.prob[i] = fill_params(a[i], pl, ws.partial + off_p, ws.t + off_t, ws.counters + off_c, ws.counters + kCtrStatus, nullptr);
        b.first[i] = (i == 0) ? 0 : b.first[i];
        b.first[i + 1] = b.first[i] + pl.n_t + pl.R * pl.SK;
        off_p += (size_t)pl.NT * pl.maxslots * a[i].M * kTileRows;
        off_t += (size_t)kDecodeMaxM * kMaxRank;
        off_c += kCtrFirstTile + 2 * pl.NT;
        smem = pl.smem > smem ? pl.smem : smem;
        heavy = heavy || pl.heavy;
    }
    const bool pdl = tune.pdl != 0;
    cudaError_t e = dispatch_variant(a[0], [&](auto bits, auto type, auto mt, auto hv, auto e4) {
        return launch_batch_variant<decltype(bits)::value, typename decltype(type)::type, decltype(mt)::value, decltype(hv)::value,
                                    decltype(e4)::value>(b, smem, pdl, s);
    }, heavy, i8);
    if (e == cudaSuccess) ++*launches;
    return e;
}

}  // namespace fbq
