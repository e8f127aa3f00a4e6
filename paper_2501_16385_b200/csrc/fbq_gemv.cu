// Streaming decode kernel (few tokens) of the FBQuant linear, sm_100a.
//
// One launch computes  y = x.dequant(Q,s,z)^T + (x.A^T).B^T  (Algorithm 1 step 6 of the paper;
// Section 4.3 fuses dequantisation, main product and up-projection and leaves t = x.A^T to a second
// launch; here t comes from a few CTAs of the same grid).  The kernel is built around what a launch
// of a few microseconds costs besides streaming its weights:
//
//   * Everything that comes from the WEIGHTS (packed codes, scales, zero points, B, A) is requested
//     before the kernel waits for the preceding kernel of its stream (programmatic dependent
//     launch); a CTA takes half an SM's shared memory at most, so the CTAs of the next launch are
//     resident and prefetching while this launch still computes.
//   * No table is built per CTA: scales and zero points of a 16-row tile arrive as they are stored
//     (two bulk copies per tile) and are converted where they are used.
//   * The weight stream is one TMA tensor copy per stage (16 groups x 16 rows of packed codes) into
//     an mbarrier ring; eight compute warps share every stage.
//
// Main CTAs (one per SM by default) own contiguous ranges of 16-row tiles.  Integer form (M <= 2):
// a code masked out of its word is an unsigned byte operand of the 8-bit integer MMA as it stands
// (four codes per register, at most one shift per word); x is fixed point per group of 128 (three
// signed base-256 digits, exact integer sums), and scale and zero point are applied per group to the
// integer sums in fp32.  At M = 1 an MMA's eight columns hold the digits of TWO groups (columns 0-2
// and 4-6), so the per-group fp32 work is done once per pair of groups.
// The epilogue warp of a CTA adds the eight warps' partial tiles (fixed order), adds t.B^T on tensor
// cores (t as two 16-bit terms, rows of B by TMA with the 128-byte swizzle), rounds once, stores y.
//
// t CTAs (the first n_t blocks of the grid): each holds a k-chunk of all rows of A (TMA, swizzled,
// requested before the wait), multiplies it with its chunk of x on tensor cores and stores its
// partial t to scratch; an arrival counter tells the main CTAs' epilogue warps when all chunks are
// there (bounded polling; FBQ_ERR_TIMEOUT instead of a hang), which then add the chunks in order.
#include <cuda.h>
#include <cudaTypedefs.h>

#include <cstdio>
#include <cstdlib>
#include <mutex>
#include <type_traits>
#include <vector>

#include "fbq_common.cuh"
#include "fbq_ptx.cuh"

namespace fbq {
namespace {
using namespace ptx;

#ifndef FBQ_GEMV_CW
#define FBQ_GEMV_CW 8
#endif
constexpr int kCW = FBQ_GEMV_CW;             // compute warps of a main CTA
constexpr int kCtasPerSm = (kCW <= 8) ? 2 : 1;   // CTAs of consecutive launches that share an SM
constexpr int kEpiWarp = kCW;                // then the epilogue warp
constexpr int kProdWarp = kCW + 1;           // and the producer warp
constexpr int kWarps = kCW + 2;
constexpr int kThreads = kWarps * 32;
constexpr int kTile = 16;                    // weight rows of a tile
constexpr int kCHG = 2 * kCW;                // quantisation groups of a stage (one pair per compute warp at M = 1)
constexpr int kMaxNS = 8, kMaxBuf = 8, kMaxB = 4, kMaxMeta = 8;
constexpr int kMaxSub = 8;                   // tiles whose t.B^T may be formed ahead of their main sums
constexpr int kTKB = 64;                     // k extent of one block of A in a t CTA (128 bytes: the swizzle span)

struct GemvParams {
    const void *x;
    const __half *scales;
    const __half *zeros;
    void *y;
    int slot_elems;     // words from one slot of tpart to the next: M * rank rounded up to whole 128-byte lines (slots
                        // that share a line make the line a hot spot: every main CTA polls it while a t CTA writes it)
    uint32_t *tpart;    // [n_t (+ 1)][M][rank] partial sums of t, one slot per t CTA (and one for their sum), each entry
                        // one word: the fp32 value with +0.0 stored as -0.0, so a word is zero exactly while it has not been written
                        // by this launch; all words are zero on entry and on exit
    int *ctr;           // [1] main CTAs that have read t; zero on entry and exit
    int *status;        // receives FBQ_ERR_TIMEOUT when a bounded wait runs out
    int M, N, K, G, rank;
    int NT;             // tiles
    int n_t, n_main;
    int t_kb;           // blocks of kTKB input channels per t CTA
    int NS, nbuf, nmeta, nb;
    int stage_bytes, meta_pitch, b_slot_bytes, b_box_cols, b_swz;
    int off_bar, off_tab, off_x, off_meta, off_seg, off_t, off_B, off_ring;
    int off_tA, off_tred;                   // t CTA: blocks of A, reduction buffer
    // 16-bit form (M >= 3): K may be cut into SK slices (CTA = row block x slice) whose partial tiles meet in scratch
    int SK, R;                              // n_main = R * SK
    int slice_groups;                       // groups per K slice (a multiple of the stage's groups; the last slice takes the rest)
    int x_pitch;                            // elements between tokens of the staged x
    int off_px, off_tf;                     // (P, X0) table; t as MMA column operands
    int off_sub;                            // t.B^T of the tiles ahead (integer form)
    float *part;                            // [tile][slice][M][16] fp32 partial tiles (SK > 1)
    int *tctr;                              // [tile] slices that have stored their partial (zero on entry and exit)
    int t_final;                            // 1: the t CTA that arrives last adds the slots into slot n_t, and the main CTAs read only that one
    uint32_t poll_limit;                    // looks at the arrival counter before giving up
    int pair;                               // 16-bit form: CTAs come in clusters of two that stage half of x each
    int test_skip_arrive;                   // test switch: t CTAs do not report their arrival
    unsigned long long *trace;              // optional phase timestamps [cta][warp][16] (tuning aid), else NULL
};

// barrier slots (8 bytes each) from off_bar
constexpr int kBarFull = 0, kBarEmpty = kMaxNS, kBarSegFull = 2 * kMaxNS, kBarSegFree = 2 * kMaxNS + kMaxBuf,
              kBarB = 2 * kMaxNS + 2 * kMaxBuf, kBarA = kBarB + kMaxB, kBarXReq = kBarA + 1, kNumBars = kBarXReq + 1;
constexpr int kEarlyStages = 1;               // weight stages requested before the loads of x are on their way

// ------------------------------------------------- integer form: codes as bytes
// A 3- or 4-bit code masked out of its word where it sits is the unsigned byte q * 2^j (j = the
// field's offset inside its byte): an operand of the 8-bit integer MMA as it stands.
//   INT4 word i:  r[2i]   = w & 0x0F0F0F0F          codes 8i+0, 8i+2, 8i+4, 8i+6
//                 r[2i+1] = w & 0xF0F0F0F0          codes 8i+1, 8i+3, 8i+5, 8i+7   (x 16)
//   INT3 word i:  r[3i]   = w & 0x0E070E07          codes 10i+0, 10i+3 (x 2), 10i+5, 10i+8 (x 2)
//                 r[3i+1] = w & 0x70387038          codes 10i+1 (x 8), 10i+4 (x 16), 10i+6 (x 8), 10i+9 (x 16)
//                 r[3i+2] = (w >> 6) & 0x02070207   codes 10i+2, bit i of code 30 (x 2), 10i+7, bit i of code 31 (x 2)
// (The three bits of the bit-sliced codes 30 and 31 are operands of their own: 36 byte slots per 32
// codes.  With and-masks alone no layout of 32 three-bit codes in three words gets by with 32 slots: a
// byte lane holds two whole fields and two spare bits, and the spare bits of different bytes cannot
// meet in one lane.)
template <int BITS> struct Slots {
    static constexpr int kRegs = (BITS == 4) ? 8 : 9;
    static constexpr int kWords = (BITS == 4) ? 4 : 3;
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

__device__ __forceinline__ float half_bits_to_float(uint32_t v) { return __half2float(__ushort_as_half((unsigned short)v)); }

// Tuning aid, compiled in with -DFBQ_GEMV_TRACE only (the marks cost code size, which this kernel feels): the
// global timer (ns) of this warp at a phase.
__device__ __forceinline__ void mark(const GemvParams &p, int slot)
{
#ifdef FBQ_GEMV_TRACE
    if (p.trace && (threadIdx.x & 31) == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
        p.trace[((size_t)blockIdx.x * kWarps + (threadIdx.x >> 5)) * 16 + slot] = t;
        if (slot == 0) {                                      // and where the CTA runs
            unsigned sm;
            asm volatile("mov.u32 %0, %%smid;" : "=r"(sm));
            p.trace[((size_t)blockIdx.x * kWarps + (threadIdx.x >> 5)) * 16 + 15] = sm;
        }
    }
#endif
}

__device__ __forceinline__ void give_up(const GemvParams &p) { atomicExch(p.status, (int)FBQ_ERR_TIMEOUT); }

// ------------------------------------------------------------------ x, integer form
// x of all K for M tokens as fixed point per group of 128: 2^e puts the group's largest |x| into
// [2^20, 2^21); per byte slot X = rint(x 2^e 2^-j) (the slot's factor undone) as three signed
// base-256 digits, X = d0 2^16 + d1 2^8 + d2 (the bytes of (X + 0x808080) ^ 0x808080).  Digit i of
// token m is MMA column 4m + i (M = 2) or 4 (group parity) + i (M = 1).  Layout in shared memory:
// 16-byte units [group][register quad 0..1][column 3m+i][lane t] (registers 4p..4p+3 of the
// unpacked codes), then one word per [group][column][lane t] for register 8 of INT3.  The table
// holds, per (group, token), two float4: (2^-e 2^16, 2^-e 2^8, sum of x, 0) for the lanes that hold
// digits 0 and 1 and (2^-e, 0, 0, 0) for the lanes that hold digit 2.  A group with a non-finite x
// gets NaN there, so that its outputs are NaN as the definition says.
template <int BITS, typename T, int M>
__device__ __forceinline__ void convert_x(const GemvParams &p, uint8_t *smem, int warp, int lane)
{
    // Two lanes share a 32-element run of x (the k range of lane t of one group): the even lane makes
    // the digits of registers 0..3, the odd lane the rest.  Each takes half of the run for the group's
    // maximum and sum (the eight lanes of a group sit side by side), and converts only the elements
    // its own slots need.
    constexpr int NR = Slots<BITS>::kRegs;
    constexpr int ncol = 3 * M;
    const T *x = static_cast<const T *>(p.x);
    float4 *s_tab = reinterpret_cast<float4 *>(smem + p.off_tab);
    uint4 *s_x8 = reinterpret_cast<uint4 *>(smem + p.off_x);
    uint32_t *s_xt = reinterpret_cast<uint32_t *>(smem + p.off_x) + (size_t)p.G * 2 * ncol * 16;
    // Every compute warp stages exactly the groups it will multiply (the pairs st * 8 + warp of every stage, the same
    // for every tile), so no warp waits for another one's part of x.
    const int G = p.G, SPT = (G + kCHG - 1) / kCHG;
    const int units = M * SPT * 2;                                          // (group, token) units of this warp, token fastest
    const int upper = lane & 1;
    // unit u of the warp: eight lanes share it
    auto locate = [&](int it, int &m, int &run, bool &valid, int &pad) {
        const int u = it * 4 + (lane >> 3);
        const int li = u / M;
        m = u - li * M;
        const int grp = kCHG * (li >> 1) + 2 * warp + (li & 1);
        valid = u < units && grp < G;
        pad = (u < units && grp >= G) ? grp : -1;                           // a group of the last stage beyond K
        run = valid ? grp * 4 + ((lane >> 1) & 3) : 0;
    };
    // All of the warp's x is requested at once, as whole 128-byte lines (every CTA of the grid reads the same x at
    // the same moment: the fewer requests per line, the shorter the queue at its L2 slice), straight into shared
    // memory: the 256 bytes of (group, token m) land at byte 256 m of that group's digit area.  A batch of four
    // units holds all tokens of its groups, and a batch writes digits only after all its lanes have read their raw
    // x, so the digits never overwrite raw x that is still needed.
    const uint32_t xarea = smem_u32(smem) + p.off_x;
    constexpr uint32_t garea = 2u * ncol * 64u;                             // bytes of one group's digit area
    const int nbatch = (units + 3) >> 2;
    for (int it = 0; it < nbatch; ++it) {
        int m, run, pad;
        bool valid;
        locate(it, m, run, valid, pad);
        if (valid) {
            const T *src = x + (size_t)m * p.K + (size_t)(run >> 2) * 128 + (lane & 7) * 8;
            const uint32_t dst = xarea + (uint32_t)(run >> 2) * garea + (uint32_t)m * 256u + (uint32_t)(lane & 7) * 16u;
            cp_async16(dst, src);
            cp_async16(dst + 128u, src + 64);
        }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(smem) + p.off_bar + 8u * kBarXReq);    // our loads of x are on their way
    cp_async_wait_all();
    __syncwarp();
#pragma unroll 1
    for (int it = 0; it < nbatch; ++it) {
        int m, run, pad;
        bool valid;
        locate(it, m, run, valid, pad);
        // The last stage is multiplied whole: its groups beyond K arrive as zero codes (the tensor copy's fill), and
        // their table entries are zero, so they add nothing whatever stands where their x would be.
        if (pad >= 0 && (lane & 7) == 0) {
            s_tab[((size_t)pad * M + m) * 2] = make_float4(0.f, 0.f, 0.f, 0.f);
            s_tab[((size_t)pad * M + m) * 2 + 1] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        uint4 xv[4];
        {
            const uint32_t src = xarea + (uint32_t)(run >> 2) * garea + (uint32_t)m * 256u + (uint32_t)(run & 3) * 64u;
#pragma unroll
            for (int i = 0; i < 4; ++i) xv[i] = valid ? lds_v4(src + 16u * i) : make_uint4(0u, 0u, 0u, 0u);
        }
        __syncwarp();                                                       // every lane holds its raw x: digits may go there
        if (it == 0) mark(p, 9);
        const uint16_t *e = reinterpret_cast<const uint16_t *>(xv);
        float xf[32];
#pragma unroll
        for (int c = 0; c < 32; ++c) {
            T xe;
            *reinterpret_cast<uint16_t *>(&xe) = e[c];
            xf[c] = ActTraits<T>::to_float(xe);                              // only those that are used below survive
        }
        float amax = 0.f, xsum = 0.f;
#pragma unroll
        for (int c = 0; c < 16; ++c) {
            const float v = upper ? xf[16 + c] : xf[c];
            amax = fmaxf(amax, fabsf(v));
            xsum += v;
        }
#pragma unroll
        for (int o = 1; o < 8; o <<= 1) {
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            xsum += __shfl_xor_sync(0xffffffffu, xsum, o);
        }
        const bool finite = (amax <= 3.0e38f) && (fabsf(xsum) <= 3.4e38f);                // false for Inf and NaN
        const uint32_t ex = min(max(__float_as_uint(amax) >> 23, 32u), 230u);           // biased exponent of the maximum
        const float xs = __uint_as_float((274u - ex) << 23);                            // 2^(20 - floor(log2 max))
        if (valid && (lane & 7) == 0) {
            const float inv = finite ? __uint_as_float((ex - 20u) << 23) : __uint_as_float(0x7fc00000u);   // 1 / xs
            float4 *row = s_tab + ((size_t)(run >> 2) * M + m) * 2;
            row[0] = make_float4(inv * 65536.f, inv * 256.f, xsum, 0.f);
            row[1] = make_float4(inv, 0.f, 0.f, 0.f);
        }
        auto make = [&](auto rbeg, auto rend) {
            constexpr int R0 = decltype(rbeg)::value, R1 = decltype(rend)::value;
            uint32_t dg[R1 - R0][3];
#pragma unroll
            for (int R = R0; R < R1; ++R) {
                uint32_t v[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    constexpr float kPow[7] = {1.f / 16.f, 1.f / 8.f, 1.f / 4.f, 1.f / 2.f, 1.f, 2.f, 4.f};
                    const float f = xs * kPow[Slots<BITS>::scale_log2(R, j) + 4];
                    // rint(x f) for |x f| < 2^22 sits in the low bits of x f + 1.5 2^23 (round to nearest even by the FMA)
                    const uint32_t X = __float_as_uint(fmaf(xf[Slots<BITS>::code(R, j)], f, 12582912.f));
                    v[j] = (X + 0x00408080u) ^ 0x00808080u;                  // low 24 bits: (X + 0x808080) ^ 0x808080
                }
                // digit i of the four slots -> one register (byte j = slot j)
                const uint32_t lo01 = __byte_perm(v[0], v[1], 0x5140), lo23 = __byte_perm(v[2], v[3], 0x5140);
                dg[R - R0][2] = __byte_perm(lo01, lo23, 0x5410);
                dg[R - R0][1] = __byte_perm(lo01, lo23, 0x7632);
                dg[R - R0][0] = __byte_perm(__byte_perm(v[0], v[1], 0x0062), __byte_perm(v[2], v[3], 0x0062), 0x5410);
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
}

// --------------------------------------------------------------- compute warps, integer form
template <int BITS, typename T, int M>
__device__ __forceinline__ bool compute_i8(const GemvParams &p, uint8_t *smem, int warp, int lane, int tile_first, int ntile)
{
    constexpr int NR = Slots<BITS>::kRegs, NW = Slots<BITS>::kWords;
    constexpr int GB = (BITS == 4) ? 64 : 48;                  // bytes of one group of one row
    constexpr int ncol = 3 * M;
    constexpr uint32_t x_gstride = 2u * ncol * 64u;            // bytes of one group's 16-byte units
    constexpr uint32_t x_chunk1 = ncol * 64u;                  // second register quad
    constexpr uint32_t xt_gstride = ncol * 16u;
    const int g = lane >> 2, tq = lane & 3;
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bars = sbase + p.off_bar;
    const int G = p.G, NS = p.NS, SPT = (G + kCHG - 1) / kCHG;

    // ---- per-lane constants.  As an MMA column, this lane is n = g: column block n >> 2 (group parity at
    // M = 1, token at M = 2), digit n & 3 (3 = no digit: reads zeros).  As an accumulator lane it holds
    // columns 2tq, 2tq+1: block tq >> 1, digits (0, 1) or (2, none).
    const int nb = g >> 2, nc = g & 3;
    const bool has_digit = nc < 3;
    const uint32_t x8 = sbase + p.off_x, xt8 = x8 + (uint32_t)G * x_gstride;
    // lanes without a digit column, and (M = 1) lanes of the other group's block, load nothing and hold zeros
    uint32_t xa, xb = 0, xt;
    uint32_t pa, pb = 0u;
    constexpr uint32_t xsa = (M == 1) ? 2u * x_gstride : x_gstride, xts = (M == 1) ? 2u * xt_gstride : xt_gstride;
    if (M == 1) {
        // pair of groups (a, b): group a in block 0, group b in block 1
        pa = (has_digit && nb == 0) ? 1u : 0u;
        pb = (has_digit && nb == 1) ? 1u : 0u;
        xa = x8 + (uint32_t)nc * 64u + tq * 16u;
        xb = xa + x_gstride;
        xt = xt8 + (uint32_t)nb * xt_gstride + (uint32_t)nc * 16u + tq * 4u;
    } else {
        pa = has_digit ? 1u : 0u;
        xa = x8 + (uint32_t)(3 * nb + nc) * 64u + tq * 16u;
        xt = xt8 + (uint32_t)(3 * nb + nc) * 16u + tq * 4u;
    }
    const uint32_t pt = has_digit ? 1u : 0u;
    const int ablk = tq >> 1, apar = tq & 1;
    const uint32_t tab = sbase + p.off_tab + (uint32_t)((M == 1 ? 0 : ablk * 2) + apar) * 16u;     // + group index * (M * 32)
    const uint32_t w_lane = sbase + p.off_ring + (uint32_t)(g * GB + tq * (GB / 4));
    const uint32_t meta0 = sbase + p.off_meta;
    const uint32_t zoff = (uint32_t)p.meta_pitch, row8 = (uint32_t)(8 * G * 2);
    float *s_seg = reinterpret_cast<float *>(smem + p.off_seg);

    auto load_words = [&](uint32_t wa, uint32_t (&wr)[NW]) {
        if constexpr (BITS == 4) {
            const uint4 v = lds_v4(wa);
            wr[0] = v.x; wr[1] = v.y; wr[2] = v.z; wr[3] = v.w;
        } else {
#pragma unroll
            for (int i = 0; i < NW; ++i) wr[i] = lds_u32(wa + 4 * i);
        }
    };
    // the first eight registers of one group's codes (rows g and g + 8) against its digits: four MMAs
    // in two independent chains
    auto mma8 = [&](int (&d0)[4], int (&d1)[4], const uint32_t (&ra)[NR], const uint32_t (&rb)[NR], const uint4 &x0, const uint4 &x1) {
        mma_u8s8(d0, ra[0], rb[0], ra[1], rb[1], x0.x, x0.y);
        mma_u8s8(d1, ra[2], rb[2], ra[3], rb[3], x0.z, x0.w);
        mma_u8s8(d0, ra[4], rb[4], ra[5], rb[5], x1.x, x1.y);
        mma_u8s8(d1, ra[6], rb[6], ra[7], rb[7], x1.z, x1.w);
    };
    // scale, zero point and the weights of the digits: integer sums of one block -> fp32
    struct Meta {
        float4 tb;
        uint32_t sg, zg, sh, zh;
    };
    auto load_meta = [&](uint32_t tabaddr, uint32_t maddr) {
        Meta m;
        m.tb = lds_f4(tabaddr);
        m.sg = lds_u16(maddr);
        m.zg = lds_u16(maddr + zoff);
        m.sh = lds_u16(maddr + row8);
        m.zh = lds_u16(maddr + row8 + zoff);
        return m;
    };
    auto scale = [&](const int (&d)[4], const Meta &m, float (&acc)[2]) {
        const float sg = half_bits_to_float(m.sg), zg = half_bits_to_float(m.zg);
        const float sh = half_bits_to_float(m.sh), zh = half_bits_to_float(m.zh);
        float fg = fmaf((float)d[1], m.tb.y, (float)d[0] * m.tb.x);
        float fh = fmaf((float)d[3], m.tb.y, (float)d[2] * m.tb.x);
        fg = fmaf(-zg, m.tb.z, fg);
        fh = fmaf(-zh, m.tb.z, fh);
        acc[0] = fmaf(sg, fg, acc[0]);
        acc[1] = fmaf(sh, fh, acc[1]);
    };

    // this warp's partial tile: add the lanes of a block (and, at M = 1, both blocks), hand it to the epilogue warp
    int dep_buf = 0;
    uint32_t dep_phase = 1u;                       // parity of the buffer's previous use; unused while dep_first
    bool dep_first = true;
    auto deposit = [&](int ts, float (&acc)[2]) -> bool {
        acc[0] += __shfl_xor_sync(0xffffffffu, acc[0], 1);
        acc[1] += __shfl_xor_sync(0xffffffffu, acc[1], 1);
        if (M == 1) {
            acc[0] += __shfl_xor_sync(0xffffffffu, acc[0], 2);
            acc[1] += __shfl_xor_sync(0xffffffffu, acc[1], 2);
        }
        const int buf = dep_buf;
        if (!dep_first && !mbar_wait(bars + 8u * (kBarSegFree + buf), dep_phase)) return false;
        if (apar == 0 && ablk < M) {
            float *dst = s_seg + ((size_t)(buf * kCW + warp) * M + ablk) * kTile;
            dst[g] = acc[0];
            dst[g + 8] = acc[1];
        }
        __syncwarp();
        mbar_arrive_if(bars + 8u * (kBarSegFull + buf), lane == 0);
        mark(p, ts == 0 ? 5 : 6);
        acc[0] = acc[1] = 0.f;
        if (++dep_buf == p.nbuf) {
            dep_buf = 0;
            dep_phase = dep_first ? 0u : dep_phase ^ 1u;
            dep_first = false;
        }
        return true;
    };

    if constexpr (M == 1) {
        // One pass = one pair of groups (a, b) of one tile: group a in column block 0, group b in block 1.
        // Software pipeline over the passes of all tiles: the packed words of the NEXT pass are loaded
        // while the MMAs of this one are in flight, and the per-group fp32 work follows those loads.
        const int total = ntile * SPT;
        const uint32_t woff = (uint32_t)(2 * warp) * (kTile * GB);
        uint32_t wa0[NW], wa1[NW], wb0[NW], wb1[NW];
        auto load_pass = [&](int slot) {
            const uint32_t wa = w_lane + (uint32_t)slot * (uint32_t)p.stage_bytes + woff;
            load_words(wa, wa0);
            load_words(wa + 8 * GB, wa1);
            load_words(wa + kTile * GB, wb0);
            load_words(wa + kTile * GB + 8 * GB, wb1);
        };
        if (total > 0) {
            if (!mbar_wait(bars + 8u * kBarFull, 0u)) return false;
            mark(p, 4);
            load_pass(0);
        }
        float acc[2] = {0.f, 0.f};
        int ts = 0, st = 0, slot = 0, nslot = (NS > 1) ? 1 : 0;
        uint32_t npar = (NS > 1) ? 0u : 1u;                           // parity of the next stage's first completion
        uint32_t mslot = meta0 + (uint32_t)(g * G * 2);
        int mi = 0;
        for (int it = 0; it < total; ++it) {
            const int pi = st * (kCHG / 2) + warp, ga = 2 * pi;
            constexpr bool live = true;                                    // groups beyond K are zero codes with a zero table entry
            Meta mt;
            int d0[4] = {0, 0, 0, 0}, d1[4] = {0, 0, 0, 0}, d2[4] = {0, 0, 0, 0}, d3[4] = {0, 0, 0, 0};
            if (live) {
                const uint32_t xpa = xa + (uint32_t)pi * xsa, xpb = xb + (uint32_t)pi * xsa;
                const uint4 xa0 = lds_v4_if(xpa, pa), xa1 = lds_v4_if(xpa + x_chunk1, pa);
                const uint4 xb0 = lds_v4_if(xpb, pb), xb1 = lds_v4_if(xpb + x_chunk1, pb);
                uint32_t tv = 0;
                if constexpr (BITS == 3) tv = lds_u32_if(xt + (uint32_t)pi * xts, pt);
                const int grp = min(ga + ablk, G - 1);
                mt = load_meta(tab + (uint32_t)(ga + ablk) * 32u, mslot + (uint32_t)grp * 2u);
                uint32_t ra[NR], rb[NR];
                Slots<BITS>::run(wa0, ra);
                Slots<BITS>::run(wa1, rb);
                mma8(d0, d1, ra, rb, xa0, xa1);
                uint32_t ta = 0, tb2 = 0;
                if constexpr (BITS == 3) {
                    ta = ra[8];
                    tb2 = rb[8];
                }
                Slots<BITS>::run(wb0, ra);
                Slots<BITS>::run(wb1, rb);
                mma8(d2, d3, ra, rb, xb0, xb1);
                if constexpr (BITS == 3) mma_u8s8(d0, ta, tb2, ra[8], rb[8], nb == 0 ? tv : 0u, nb == 0 ? 0u : tv);
            }
            // the next pass's words, while the MMAs run
            int nst = st + 1, nts = ts;
            if (nst == SPT) {
                nst = 0;
                ++nts;
            }
            if (it + 1 < total && !mbar_wait(bars + 8u * (kBarFull + nslot), npar)) return false;
            load_pass(nslot);                                               // after the last pass: words that nobody uses
            if (live) {
#pragma unroll
                for (int i = 0; i < 4; ++i) d0[i] = (d0[i] + d1[i]) + (d2[i] + d3[i]);
                scale(d0, mt, acc);
            }
            __syncwarp();
            mbar_arrive_if(bars + 8u * (kBarEmpty + slot), lane == 0);
            if (nts != ts) {
                if (!deposit(ts, acc)) return false;
                if (++mi == p.nmeta) mi = 0;
                mslot = meta0 + (uint32_t)mi * 2u * zoff + (uint32_t)(g * G * 2);
            }
            st = nst;
            ts = nts;
            slot = nslot;
            if (++nslot == NS) {
                nslot = 0;
                npar ^= 1u;
            }
        }
    } else {
        int slot = 0, mi = 0;
        uint32_t par = 0u;
        bool first = true;
        for (int ts = 0; ts < ntile; ++ts) {
            float acc[2] = {0.f, 0.f};
            const uint32_t mslot = meta0 + (uint32_t)mi * 2u * zoff + (uint32_t)(g * G * 2);
            if (++mi == p.nmeta) mi = 0;
            for (int st = 0; st < SPT; ++st) {
                if (!mbar_wait(bars + 8u * (kBarFull + slot), par)) return false;
                if (first) mark(p, 4);
                first = false;
                const uint32_t ws = w_lane + (uint32_t)slot * (uint32_t)p.stage_bytes;
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int gi = 2 * warp + u, grp = st * kCHG + gi;
                    const uint32_t wa = ws + (uint32_t)gi * (kTile * GB);
                    uint32_t w0[NW], w1[NW], ra[NR], rb[NR];
                    load_words(wa, w0);
                    load_words(wa + 8 * GB, w1);
                    const uint32_t xp = xa + (uint32_t)grp * xsa;
                    const uint4 x0 = lds_v4_if(xp, pa), x1 = lds_v4_if(xp + x_chunk1, pa);
                    uint32_t tv = 0;
                    if constexpr (BITS == 3) tv = lds_u32_if(xt + (uint32_t)grp * xts, pt);
                    const Meta mt = load_meta(tab + (uint32_t)grp * 64u, mslot + (uint32_t)min(grp, G - 1) * 2u);
                    int d0[4] = {0, 0, 0, 0}, d1[4] = {0, 0, 0, 0};
                    Slots<BITS>::run(w0, ra);
                    Slots<BITS>::run(w1, rb);
                    mma8(d0, d1, ra, rb, x0, x1);
                    if constexpr (BITS == 3) mma_u8s8(d1, ra[8], rb[8], 0u, 0u, tv, 0u);
#pragma unroll
                    for (int i = 0; i < 4; ++i) d0[i] += d1[i];
                    scale(d0, mt, acc);
                }
                __syncwarp();
                mbar_arrive_if(bars + 8u * (kBarEmpty + slot), lane == 0);
                if (++slot == NS) {
                    slot = 0;
                    par ^= 1u;
                }
            }
            if (!deposit(ts, acc)) return false;
        }
    }
    return true;
}

// ------------------------------------------------------------------------ producer
__device__ __forceinline__ bool produce(const GemvParams &p, uint8_t *smem, const CUtensorMap *wmap, int tile_first, int ntile,
                                        int g_begin = 0, int g_count = -1, int chg = kCHG)
{
    const uint32_t sbase = smem_u32(smem), bars = sbase + p.off_bar;
    const uint32_t ring = sbase + p.off_ring, meta0 = sbase + p.off_meta;
    if (g_count < 0) g_count = p.G;
    const int SPT = (g_count + chg - 1) / chg, NS = p.NS;
    int it = 0;
    for (int ts = 0; ts < ntile; ++ts) {
        const int tile = tile_first + ts;
        const int rows = min(kTile, p.N - tile * kTile);
        const uint32_t mbytes = (uint32_t)rows * (uint32_t)p.G * 2u;
        for (int st = 0; st < SPT; ++st, ++it) {
            const int slot = it % NS;
            // Until the compute warps have put their loads of x (which everything waits for) into the memory
            // system, keep the prefetch shallow: x must not queue behind weights that cannot be used before it.
            if (it == kEarlyStages && !mbar_wait_idle(bars + 8u * kBarXReq, 0u)) return false;
            if (it >= NS && !mbar_wait_idle(bars + 8u * (kBarEmpty + slot), (uint32_t)(it / NS - 1) & 1u)) return false;
            const uint32_t full = bars + 8u * (kBarFull + slot);
            mbar_expect_tx(full, (uint32_t)p.stage_bytes + (st == 0 ? 2u * mbytes : 0u));
            // one box of 16 groups x 16 rows (rows past N and groups past G arrive as zeros)
            tma_load_3d(ring + (uint32_t)slot * (uint32_t)p.stage_bytes, wmap, 0, tile * kTile, g_begin + st * chg, full);
            if (it == 0) mark(p, 3);
            if (st == 0) {
                const uint32_t ms = meta0 + (uint32_t)(ts % p.nmeta) * 2u * (uint32_t)p.meta_pitch;
                const size_t off = (size_t)tile * kTile * p.G;
                bulk_g2s(ms, p.scales + off, mbytes, full);
                bulk_g2s(ms + (uint32_t)p.meta_pitch, p.zeros + off, mbytes, full);
            }
        }
    }
    mark(p, 6);
    return true;
}

// Before the wait for the preceding kernel: up to 64 lines of x per CTA are asked into L2 (the CTAs of a launch
// start at different lines, so that together they cover a large x).  The preceding kernel may still be writing x:
// its stores meet the lines in L2 then.  Saves the compute warps the cold miss on their first read of x.
__device__ __forceinline__ void prefetch_x(const GemvParams &p, int cta, int lane, int elem_bytes)
{
    const int nlines = (int)(((size_t)p.M * p.K * elem_bytes + 127) / 128);
    const char *x = static_cast<const char *>(p.x);
    for (int j = lane; j < min(nlines, 64); j += 32) prefetch_l2(x + (size_t)((cta * 64 + j) % nlines) * 128);
}

// ------------------------------------------------------------------------ epilogue warp
// Swizzled byte offset inside a tile that TMA wrote with the 32-, 64- or 128-byte swizzle
// (mask 1, 3, 7): the 16-byte unit index is XOR-ed with the 128-byte line index.
__device__ __forceinline__ uint32_t swz(uint32_t off, uint32_t mask) { return off ^ (((off >> 7) & mask) << 4); }

// An entry of a t slot is the fp32 value itself, with +0.0 stored as -0.0: the word is never zero once written, so
// value and "written" travel in one 4-byte store, a reader may fetch four entries with one 16-byte load, add them as
// they are (-0.0 adds like +0.0, and a sum that starts at +0.0 stays +0.0) and check each word by itself; memory that
// is zero means "not yet".
constexpr uint32_t kTNone = 0x80000000u;                     // -0.0: what a slot that does not exist reads as
__device__ __forceinline__ uint32_t t_enc(float v) { const uint32_t w = __float_as_uint(v); return w ? w : kTNone; }
__device__ __forceinline__ uint32_t t_min(uint32_t m, const uint4 &w) { return __vimin3_u32(m, __vimin3_u32(w.x, w.y, w.z), w.w); }

// One look at exactly eight t slots with at most 128 entries: straight-line code, a lane takes four consecutive
// entries and has its eight 16-byte loads in flight at once (the common shapes: the looks are what a main CTA's
// epilogue waits with, and a lean look is a fast look).  Adds the slots in slot order into s_t, returns whether
// every entry was there; amax = largest |sum|.
__device__ __forceinline__ bool look8(const uint32_t *slots, size_t slot_elems, int nent, int lane, float *s_t, float &amax)
{
    const int nq = nent >> 2, q = min(lane, nq - 1);          // lanes past the last four entries repeat them (and do not store)
    uint4 pv[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) pv[u] = __ldcg(reinterpret_cast<const uint4 *>(slots + (size_t)u * slot_elems) + q);
    uint32_t mn = 0xFFFFFFFFu;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        mn = t_min(mn, pv[u]);
        v.x += __uint_as_float(pv[u].x);
        v.y += __uint_as_float(pv[u].y);
        v.z += __uint_as_float(pv[u].z);
        v.w += __uint_as_float(pv[u].w);
    }
    if (lane < nq) *reinterpret_cast<float4 *>(s_t + 4 * lane) = v;
    amax = fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w)));
    return mn != 0u;
}

// The same for any number of slots and entries: four entries x eight slots in flight per lane, added in slot order.
__device__ __forceinline__ bool look_slots(const uint32_t *tpart, size_t slot_elems, int s_first, int s_end, int nent, int lane,
                                           float *s_t, float &amax)
{
    uint32_t mn = 0xFFFFFFFFu;
    amax = 0.f;
    for (int q = lane; 4 * q < nent; q += 32) {
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int c0 = s_first; c0 < s_end; c0 += 8) {
            uint4 pa[8];
#pragma unroll
            for (int u = 0; u < 8; ++u)
                pa[u] = (c0 + u < s_end) ? __ldcg(reinterpret_cast<const uint4 *>(tpart + (size_t)(c0 + u) * slot_elems) + q)
                                         : make_uint4(kTNone, kTNone, kTNone, kTNone);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                mn = t_min(mn, pa[u]);
                v.x += __uint_as_float(pa[u].x);
                v.y += __uint_as_float(pa[u].y);
                v.z += __uint_as_float(pa[u].z);
                v.w += __uint_as_float(pa[u].w);
            }
        }
        *reinterpret_cast<float4 *>(s_t + 4 * q) = v;
        amax = fmaxf(amax, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
    }
    return mn != 0u;
}

template <typename T, bool RANKED>
__device__ __forceinline__ bool epilogue(const GemvParams &p, uint8_t *smem, const CUtensorMap *bmap, int lane, int tile_first, int ntile)
{
    const int g = lane >> 2, tq = lane & 3;
    const uint32_t sbase = smem_u32(smem), bars = sbase + p.off_bar;
    const uint32_t bring = sbase + p.off_B;
    const int rank = RANKED ? p.rank : 0, M = p.M, nkb = rank / 16;
    const int nbox = (rank + 63) / 64;
    const uint32_t box_bytes = (uint32_t)kTile * (uint32_t)p.b_box_cols * 2u;
    auto request_b = [&](int ts, int slot) {
        const uint32_t bar = bars + 8u * (kBarB + slot);
        mbar_expect_tx(bar, (uint32_t)nbox * box_bytes);
        for (int b = 0; b < nbox; ++b)
            tma_load_2d(bring + (uint32_t)slot * (uint32_t)p.b_slot_bytes + (uint32_t)b * box_bytes, bmap, b * 64,
                        (tile_first + ts) * kTile, bar);
    };
    if (RANKED && lane == 0)
        for (int ts = 0; ts < min(ntile, p.nb); ++ts) request_b(ts, ts);   // rows of B are weights: before the wait
    prefetch_x(p, (int)blockIdx.x - p.n_t, lane, (int)sizeof(T));
    // Everything this warp does per tile runs alone on its latencies, so what does not depend on the tile is done
    // once, and before the wait: this lane's (swizzled) byte offsets into a tile of B, as MMA row fragments of the
    // four 16-wide blocks of a 64-column box.
    const uint32_t smask = (uint32_t)p.b_swz, pitch = (uint32_t)p.b_box_cols * 2u;
    uint32_t aoff[4][4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const uint32_t c0 = (uint32_t)(q * 32 + tq * 4);                  // bytes into the row
        const uint32_t o0 = (uint32_t)g * pitch + c0, o1 = o0 + 8u * pitch;
        aoff[q][0] = swz(o0, smask);
        aoff[q][1] = swz(o1, smask);
        aoff[q][2] = swz(o0 + 16u, smask);
        aoff[q][3] = swz(o1 + 16u, smask);
    }

    uint32_t *s_tf = reinterpret_cast<uint32_t *>(smem + p.off_tf);      // t as MMA column operands [rank block][lane][2]
    if constexpr (RANKED) {
        for (int i = lane; i < nkb * 64; i += 32) s_tf[i] = 0u;
        __syncwarp();
    }

    pdl_wait();
    mark(p, 2);

    // ---- t: wait for the t CTAs, add their chunks in order, keep t as MMA column operands ----
    float isc = 1.f;
    if constexpr (RANKED) {
        // Look at the t CTAs' slots themselves until every entry carries this launch's tag (bounded), adding
        // the chunks in slot order.
        float *s_t = reinterpret_cast<float *>(smem + p.off_t);
        float amax = 0.f;
        const size_t slot_elems = (size_t)p.slot_elems;
        const int s_first = p.t_final ? p.n_t : 0, s_end = p.t_final ? p.n_t + 1 : p.n_t;    // the slots to add (or the one that holds their sum)
        bool ok = false;
        for (uint32_t look = 0; look < p.poll_limit && !ok; ++look) {
            bool all = true;
            amax = 0.f;
            if (s_end - s_first == 8 && M * rank <= 128)
                all = look8(p.tpart + (size_t)s_first * slot_elems, slot_elems, M * rank, lane, s_t, amax);
            else
                all = look_slots(p.tpart, slot_elems, s_first, s_end, M * rank, lane, s_t, amax);
            ok = __all_sync(0xffffffffu, all);
            if (!ok && look > 256) __nanosleep(64);
        }
        if (!ok) return false;
        // Tell that this CTA has read t (nobody waits for the add; a t CTA clears up once all have told).
        if (lane == 0) atomicAdd(p.ctr + 1, 1);
        // the largest |sum| of the warp: non-negative floats order like their bit patterns, so one integer reduction does
        // (a NaN or Inf among them ends up at the top and is clamped below, as before)
        const uint32_t amax_bits = __reduce_max_sync(0xffffffffu, __float_as_uint(amax));
        __syncwarp();
        // a power of two that puts the largest |t| near 2^14 keeps both terms inside fp16
        const uint32_t ex = min(max(amax_bits >> 23, 1u), 254u);
        const uint32_t sb = min(max(268u - ex, 1u), 254u);
        const float sc = __uint_as_float(sb << 23);
        isc = __uint_as_float((254u - sb) << 23);
        // t as MMA column operands: column 2 tok holds the rounded values of token tok, column 2 tok + 1 what the
        // rounding left; a lane takes pairs of consecutive rank indices (all lanes busy: this runs on the critical
        // path of the launch), the columns beyond the tokens were set to zero before the wait.
        const int half_rank = rank >> 1;
        for (int idx = lane; idx < M * half_rank; idx += 32) {
            const int tok = idx / half_rank, k0 = 2 * (idx - tok * half_rank);
            const float2 tv = *reinterpret_cast<const float2 *>(s_t + tok * rank + k0);
            const float v0 = tv.x * sc, v1 = tv.y * sc;
            const T h0 = ActTraits<T>::from_float(v0), h1 = ActTraits<T>::from_float(v1);
            const T l0 = ActTraits<T>::from_float(v0 - ActTraits<T>::to_float(h0));
            const T l1 = ActTraits<T>::from_float(v1 - ActTraits<T>::to_float(h1));
            const uint32_t pk_hi = (uint32_t)(*reinterpret_cast<const uint16_t *>(&h0)) | ((uint32_t)(*reinterpret_cast<const uint16_t *>(&h1)) << 16);
            const uint32_t pk_lo = (uint32_t)(*reinterpret_cast<const uint16_t *>(&l0)) | ((uint32_t)(*reinterpret_cast<const uint16_t *>(&l1)) << 16);
            const int kb = k0 >> 4, h = (k0 >> 3) & 1, q = (k0 & 7) >> 1;      // rank block, half of it, lane's quarter
            s_tf[((size_t)kb * 32 + (2 * tok) * 4 + q) * 2 + h] = pk_hi;
            s_tf[((size_t)kb * 32 + (2 * tok + 1) * 4 + q) * 2 + h] = pk_lo;
        }
        __syncwarp();
    }

    mark(p, 3);
    const float *s_seg = reinterpret_cast<const float *>(smem + p.off_seg);
    T *y = static_cast<T *>(p.y);
    // t.B^T of a tile needs t and the tile's rows of B only, so it is formed ahead of the tile's main sums, while the
    // compute warps are still at them: what is left to do when a tile's sums arrive is short.
    float2 *s_sub = reinterpret_cast<float2 *>(smem + p.off_sub) + lane;       // [tile % kMaxSub][lane]: rows g and g + 8
    int nsub = 0, sb_slot = 0;
    uint32_t sb_par = 0u;
    // t as column operands of the first four rank blocks stays in registers for all tiles
    uint32_t tfr[4][2] = {{0u, 0u}, {0u, 0u}, {0u, 0u}, {0u, 0u}};
    if constexpr (RANKED) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            tfr[q][0] = q < nkb ? s_tf[((size_t)q * 32 + lane) * 2] : 0u;
            tfr[q][1] = q < nkb ? s_tf[((size_t)q * 32 + lane) * 2 + 1] : 0u;
        }
    }
    auto sub_tile = [&](int j) -> bool {
        if (!mbar_wait(bars + 8u * (kBarB + sb_slot), sb_par)) return false;
        const uint32_t bt = bring + (uint32_t)sb_slot * (uint32_t)p.b_slot_bytes;
        // four 16-wide blocks of the rank at a time: their rows of B first, then the MMAs (two chains)
        float d[4] = {0.f, 0.f, 0.f, 0.f}, e[4] = {0.f, 0.f, 0.f, 0.f};
        {
            uint32_t af[4][4];
#pragma unroll
            for (int q = 0; q < 4; ++q)
#pragma unroll
                for (int r = 0; r < 4; ++r) af[q][r] = q < nkb ? lds_u32(bt + aoff[q][r]) : 0u;
            Mma16<T>::run(d, af[0][0], af[0][1], af[0][2], af[0][3], tfr[0][0], tfr[0][1]);
            Mma16<T>::run(e, af[1][0], af[1][1], af[1][2], af[1][3], tfr[1][0], tfr[1][1]);
            Mma16<T>::run(d, af[2][0], af[2][1], af[2][2], af[2][3], tfr[2][0], tfr[2][1]);
            Mma16<T>::run(e, af[3][0], af[3][1], af[3][2], af[3][3], tfr[3][0], tfr[3][1]);
        }
        if (nkb > 4) {                                                          // rank above 64: the second box
            const uint32_t bx = bt + box_bytes, tf_lane = sbase + p.off_tf + (uint32_t)lane * 8u;
            uint32_t af[4][4], tf[4][2];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const bool on = 4 + q < nkb;
#pragma unroll
                for (int r = 0; r < 4; ++r) af[q][r] = on ? lds_u32(bx + aoff[q][r]) : 0u;
                tf[q][0] = on ? lds_u32(tf_lane + (uint32_t)((4 + q) * 32) * 8u) : 0u;
                tf[q][1] = on ? lds_u32(tf_lane + (uint32_t)((4 + q) * 32) * 8u + 4u) : 0u;
            }
            Mma16<T>::run(d, af[0][0], af[0][1], af[0][2], af[0][3], tf[0][0], tf[0][1]);
            Mma16<T>::run(e, af[1][0], af[1][1], af[1][2], af[1][3], tf[1][0], tf[1][1]);
            Mma16<T>::run(d, af[2][0], af[2][1], af[2][2], af[2][3], tf[2][0], tf[2][1]);
            Mma16<T>::run(e, af[3][0], af[3][1], af[3][2], af[3][3], tf[3][0], tf[3][1]);
        }
        s_sub[(size_t)(j & (kMaxSub - 1)) * 32] = make_float2((d[0] + d[1]) + (e[0] + e[1]), (d[2] + d[3]) + (e[2] + e[3]));
        __syncwarp();
        if (lane == 0 && j + p.nb < ntile) request_b(j + p.nb, sb_slot);        // the slot just read
        if (++sb_slot == p.nb) {
            sb_slot = 0;
            sb_par ^= 1u;
        }
        return true;
    };
    int buf = 0;
    uint32_t seg_par = 0u;
    for (int ts = 0; ts < ntile; ++ts) {
        const uint32_t seg_bar = bars + 8u * (kBarSegFull + buf);
        if constexpr (RANKED) {
            while (nsub < ntile && nsub - ts < kMaxSub) {
                if (nsub > ts && __any_sync(0xffffffffu, mbar_try_wait(seg_bar, seg_par))) break;     // this tile's sums are there: finish it first
                if (!sub_tile(nsub)) return false;
                ++nsub;
            }
        }
        if (!mbar_wait_idle_warp(seg_bar, seg_par)) return false;
        if (ts == 0) mark(p, 4);
        float vg = 0.f, vh = 0.f;
        if (tq < M) {
            // the eight warps' partial sums, added pairwise in a fixed order (a short chain: this warp runs alone on its latencies)
            const float *src = s_seg + ((size_t)buf * kCW * M + tq) * kTile;
            float pg[kCW], ph[kCW];
#pragma unroll
            for (int w = 0; w < kCW; ++w) {
                pg[w] = src[(size_t)w * M * kTile + g];
                ph[w] = src[(size_t)w * M * kTile + g + 8];
            }
#pragma unroll
            for (int span = 1; span < kCW; span *= 2)
#pragma unroll
                for (int w = 0; w + span < kCW; w += 2 * span) {
                    pg[w] += pg[w + span];
                    ph[w] += ph[w + span];
                }
            vg = pg[0];
            vh = ph[0];
        }
        __syncwarp();
        mbar_arrive_if(bars + 8u * (kBarSegFree + buf), lane == 0);
        if constexpr (RANKED) {
            const float2 sb = s_sub[(size_t)(ts & (kMaxSub - 1)) * 32];
            vg = fmaf(sb.x, isc, vg);
            vh = fmaf(sb.y, isc, vh);
        }
        const int n = (tile_first + ts) * kTile + g;
        if (tq < M) {
            if (n < p.N) y[(size_t)tq * p.N + n] = ActTraits<T>::from_float(vg);
            if (n + 8 < p.N) y[(size_t)tq * p.N + n + 8] = ActTraits<T>::from_float(vh);
        }
        mark(p, ts == 0 ? 5 : 6);
        if (++buf == p.nbuf) {
            buf = 0;
            seg_par ^= 1u;
        }
    }
    return true;
}


// =============================================================== 16-bit form (3 <= M <= 16)
// Codes become packed 16-bit floats with one LOP3 per pair ("bias-free" unpack): a field at bit p of a
// 16-bit half, OR-ed into the mantissa of MAGIC = 1024 (fp16) or 128 (bf16), is MAGIC + 2^p q.  Nothing is
// spent per element on removing MAGIC, 2^p or the zero point: x is staged divided by 2^p (exact) and
// permuted into the order the unpacker produces, so the MMA yields sum x q + sum (MAGIC / 2^p) x; the second
// sum (P) and sum x (X0) depend on token and group only and are tabulated when x is staged, and a group
// contributes s (mma - P) - (s z) X0.
//   INT4: h[4i+e]  = codes (8i+e , 8i+e+4)  of word i          (i = 0..3, e = 0..3)
//   INT3: h[5i+f]  = codes (10i+f, 10i+5+f) of word i          (i = 0..2, f = 0..4);  h[15] = codes (30, 31)
__device__ __forceinline__ uint32_t lop3_and_or(uint32_t a, uint32_t mask, uint32_t orv)
{
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(a), "r"(mask), "r"(orv));   // (a & mask) | orv
    return r;
}
template <int BITS, typename T> struct Unpack16;
template <> struct Unpack16<4, __half> {
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
template <> struct Unpack16<4, __nv_bfloat16> {
    static constexpr float kMagic = 128.f;                     // 0x4300 | q is 128 + q in bf16 (7 mantissa bits)
    static __device__ __forceinline__ int div_log2(int) { return 0; }
    static __device__ __forceinline__ void run(const uint32_t *w, uint32_t *h)
    {
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) h[4 * i + e] = lop3_and_or(w[i] >> (4 * e), 0x000F000Fu, 0x43004300u);
    }
};
template <> struct Unpack16<3, __half> {
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
template <> struct Unpack16<3, __nv_bfloat16> {
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
// Position of code c (0..31) of a lane's 32-code run in that order: 2 * h_index + (0 = low half, 1 = high half).
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
constexpr int kCHGW = 8;                     // groups of a stage in the 16-bit form: one per compute warp
static_assert(kCHGW == kCW, "the 16-bit form gives every compute warp one group of a stage");

// x of this CTA's K slice (groups g_begin .. g_begin + g_count) for M tokens: per token and group the sixteen
// fragment-order pairs of a lane's run as 16-byte units [h_index / 4][lane t][h_index % 4]; (P, X0) per (group, token).
template <int BITS, typename T, int MT>
__device__ __forceinline__ void convert_x16(const GemvParams &p, uint8_t *smem, int g_begin, int g_count)
{
    const int tid = threadIdx.x, lane = tid & 31, nthr = kCW * 32;
    T *s_x = reinterpret_cast<T *>(smem + p.off_x);
    float2 *s_px = reinterpret_cast<float2 *>(smem + p.off_px);
    const T *x = static_cast<const T *>(p.x);
    // In a pair (cluster of two CTAs with the same x) this CTA converts every other group and stores the result into
    // both CTAs' shared memory: every CTA of the grid reads all of x from L2 otherwise, which is what staging costs.
    const int crank = p.pair ? (int)cluster_ctarank() : 0, cstep = p.pair ? 2 : 1;
    const int my_groups = (g_count - crank + cstep - 1) / cstep;             // groups crank, crank + cstep, ...
    const int runs_per_tok = my_groups * 4, nruns = p.M * runs_per_tok;      // multiples of 4
    const uint32_t peer_x = p.pair ? mapa_shared(smem_u32(s_x), (uint32_t)(crank ^ 1)) : 0u;
    const uint32_t peer_px = p.pair ? mapa_shared(smem_u32(s_px), (uint32_t)(crank ^ 1)) : 0u;
    constexpr int mp = 8 * MT;                                               // token slots of the (P, X0) table
    for (int i = tid; i < g_count * mp; i += nthr)                           // tokens beyond M contribute nothing
        if (i % mp >= p.M) s_px[i] = make_float2(0.f, 0.f);
    auto fetch = [&](int base, uint4 (&v)[4]) {
        const int idx = base + tid;
        const bool valid = idx < nruns;
        const int m = valid ? idx / runs_per_tok : 0, mr = valid ? idx - m * runs_per_tok : 0;
        const int run = ((mr >> 2) * cstep + crank) * 4 + (mr & 3);         // run of the slice: group, quarter
        const uint4 *src = reinterpret_cast<const uint4 *>(x + (size_t)m * p.K + (size_t)g_begin * kGroupFast + run * 32);
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] = valid ? __ldcg(src + i) : make_uint4(0u, 0u, 0u, 0u);
    };
    uint4 xn[4];
    fetch(0, xn);
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(smem) + p.off_bar + 8u * kBarXReq);   // our loads of x are on their way
#pragma unroll 1
    for (int base = 0; base < nruns; base += nthr) {
        const int idx = base + tid;                                          // whole quads are valid or not
        const bool valid = idx < nruns;
        const int m = valid ? idx / runs_per_tok : 0, mr = valid ? idx - m * runs_per_tok : 0;
        const int run = ((mr >> 2) * cstep + crank) * 4 + (mr & 3);
        uint4 xv[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) xv[i] = xn[i];
        if (base + nthr < nruns) fetch(base + nthr, xn);                     // the next batch's loads, before this batch's work
        const uint16_t *e = reinterpret_cast<const uint16_t *>(xv);
        uint32_t h[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) h[i] = 0u;
        float psum = 0.f, xsum = 0.f;
#pragma unroll
        for (int c = 0; c < 32; ++c) {
            const int pos = frag_pos<BITS>(c);                               // folds to a constant
            T xe;
            *reinterpret_cast<uint16_t *>(&xe) = e[c];
            const float xf = ActTraits<T>::to_float(xe);
            // exact division by the field weight (a power of two; up to fp16 underflow).  P is summed from the
            // stored value, so the MMA's bias term cancels exactly.
            const T xs = ActTraits<T>::from_float(xf * (1.f / (float)(1 << Unpack16<BITS, T>::div_log2(c))));
            h[pos >> 1] |= (uint32_t)(*reinterpret_cast<const uint16_t *>(&xs)) << (16 * (pos & 1));
            psum = fmaf(Unpack16<BITS, T>::kMagic, ActTraits<T>::to_float(xs), psum);
            xsum += xf;
        }
        if (valid) {
            const size_t eoff = (size_t)m * p.x_pitch + (run >> 2) * kGroupFast;    // elements into the staged x
            uint4 *dst = reinterpret_cast<uint4 *>(s_x + eoff);
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
                const uint4 v = make_uint4(h[4 * q4], h[4 * q4 + 1], h[4 * q4 + 2], h[4 * q4 + 3]);
                dst[q4 * 4 + (run & 3)] = v;
                if (p.pair) st_cluster_v4(peer_x + (uint32_t)(eoff * 2) + (uint32_t)(q4 * 4 + (run & 3)) * 16u, v);
            }
        }
        // the four runs of one (token, group) sit in four consecutive lanes
        psum += __shfl_xor_sync(0xffffffffu, psum, 1);
        xsum += __shfl_xor_sync(0xffffffffu, xsum, 1);
        psum += __shfl_xor_sync(0xffffffffu, psum, 2);
        xsum += __shfl_xor_sync(0xffffffffu, xsum, 2);
        if (valid && (run & 3) == 0) {
            s_px[(run >> 2) * mp + m] = make_float2(psum, xsum);
            if (p.pair) st_cluster_f2(peer_px + (uint32_t)((run >> 2) * mp + m) * 8u, make_float2(psum, xsum));
        }
    }
}

// Compute warps of the 16-bit form: stages of eight groups, one group per warp; MT blocks of eight tokens.
template <int BITS, typename T, int MT>
__device__ __forceinline__ bool compute_w16(const GemvParams &p, uint8_t *smem, int warp, int lane, int ntile, int g_begin, int g_count)
{
    constexpr int NW = (BITS == 4) ? 4 : 3;
    constexpr int GB = (BITS == 4) ? 64 : 48;
    const int g = lane >> 2, tq = lane & 3;
    const uint32_t sbase = smem_u32(smem), bars = sbase + p.off_bar;
    const int G = p.G, NS = p.NS, M = p.M, SPT = (g_count + kCHGW - 1) / kCHGW;
    const uint32_t w_lane = sbase + p.off_ring + (uint32_t)(warp * (kTile * GB) + g * GB + tq * (GB / 4));
    const uint32_t meta0 = sbase + p.off_meta, zoff = (uint32_t)p.meta_pitch, row8 = (uint32_t)(8 * G * 2);
    const uint32_t px_lane = sbase + p.off_px + (uint32_t)(2 * tq) * 8u;
    const uint32_t x_lane = sbase + p.off_x + (uint32_t)tq * 16u;
    const uint32_t x_tok = (uint32_t)p.x_pitch * 2u;
    float *s_seg = reinterpret_cast<float *>(smem + p.off_seg);
    int slot = 0, mi = 0, buf = 0;
    uint32_t par = 0u, dphase = 1u;
    bool first = true, dfirst = true;
    for (int ts = 0; ts < ntile; ++ts) {
        float acc[MT][4];
#pragma unroll
        for (int b = 0; b < MT; ++b) acc[b][0] = acc[b][1] = acc[b][2] = acc[b][3] = 0.f;
        const uint32_t mslot = meta0 + (uint32_t)mi * 2u * zoff + (uint32_t)(g * G * 2);
        if (++mi == p.nmeta) mi = 0;
        for (int st = 0; st < SPT; ++st) {
            if (!mbar_wait(bars + 8u * (kBarFull + slot), par)) return false;
            if (first) mark(p, 4);
            first = false;
            const int gl = st * kCHGW + warp;                          // group of the slice
            if (gl < g_count) {
                const uint32_t wa = w_lane + (uint32_t)slot * (uint32_t)p.stage_bytes;
                uint32_t w0[NW], w1[NW];
                if constexpr (BITS == 4) {
                    const uint4 va = lds_v4(wa), vb = lds_v4(wa + 8 * GB);
                    w0[0] = va.x; w0[1] = va.y; w0[2] = va.z; w0[3] = va.w;
                    w1[0] = vb.x; w1[1] = vb.y; w1[2] = vb.z; w1[3] = vb.w;
                } else {
#pragma unroll
                    for (int i = 0; i < NW; ++i) {
                        w0[i] = lds_u32(wa + 4 * i);
                        w1[i] = lds_u32(wa + 8 * GB + 4 * i);
                    }
                }
                const uint32_t ma = mslot + (uint32_t)(g_begin + gl) * 2u;
                const float sg = half_bits_to_float(lds_u16(ma)), zg = half_bits_to_float(lds_u16(ma + zoff));
                const float sh = half_bits_to_float(lds_u16(ma + row8)), zh = half_bits_to_float(lds_u16(ma + row8 + zoff));
                const float szg = sg * zg, szh = sh * zh;
                uint32_t ha[16], hb[16];
                Unpack16<BITS, T>::run(w0, ha);
                Unpack16<BITS, T>::run(w1, hb);
#pragma unroll
                for (int b = 0; b < MT; ++b) {
                    // (P, X0) of tokens 8b + 2tq and 8b + 2tq + 1 for this group; one MMA chain starts at -P
                    const float4 px = lds_f4(px_lane + (uint32_t)(gl * 8 * MT + 8 * b) * 8u);
                    float t0[4] = {-px.x, -px.z, -px.x, -px.z}, t1[4] = {0.f, 0.f, 0.f, 0.f};
                    const int token = 8 * b + g;                        // as an MMA column
                    const uint32_t xg = x_lane + (uint32_t)token * x_tok + (uint32_t)gl * (kGroupFast * 2);
                    const uint32_t on = token < M ? 1u : 0u;
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        const uint4 xv = lds_v4_if(xg + (uint32_t)q4 * 64u, on);
                        if (q4 & 1) {
                            Mma16<T>::run(t1, ha[4 * q4 + 0], hb[4 * q4 + 0], ha[4 * q4 + 1], hb[4 * q4 + 1], xv.x, xv.y);
                            Mma16<T>::run(t1, ha[4 * q4 + 2], hb[4 * q4 + 2], ha[4 * q4 + 3], hb[4 * q4 + 3], xv.z, xv.w);
                        } else {
                            Mma16<T>::run(t0, ha[4 * q4 + 0], hb[4 * q4 + 0], ha[4 * q4 + 1], hb[4 * q4 + 1], xv.x, xv.y);
                            Mma16<T>::run(t0, ha[4 * q4 + 2], hb[4 * q4 + 2], ha[4 * q4 + 3], hb[4 * q4 + 3], xv.z, xv.w);
                        }
                    }
                    // s (mma - P) - (s z) X0
                    acc[b][0] = fmaf(-szg, px.y, fmaf(sg, t0[0] + t1[0], acc[b][0]));
                    acc[b][1] = fmaf(-szg, px.w, fmaf(sg, t0[1] + t1[1], acc[b][1]));
                    acc[b][2] = fmaf(-szh, px.y, fmaf(sh, t0[2] + t1[2], acc[b][2]));
                    acc[b][3] = fmaf(-szh, px.w, fmaf(sh, t0[3] + t1[3], acc[b][3]));
                }
            }
            __syncwarp();
            mbar_arrive_if(bars + 8u * (kBarEmpty + slot), lane == 0);
            if (++slot == NS) {
                slot = 0;
                par ^= 1u;
            }
        }
        // ---- this warp's partial tile [token][16 rows] for the epilogue warp ----
        if (!dfirst && !mbar_wait(bars + 8u * (kBarSegFree + buf), dphase)) return false;
        float *dst = s_seg + (size_t)(buf * kCW + warp) * M * kTile;
#pragma unroll
        for (int b = 0; b < MT; ++b) {
            const int t0 = 8 * b + 2 * tq;
            if (t0 < M) {
                dst[t0 * kTile + g] = acc[b][0];
                dst[t0 * kTile + g + 8] = acc[b][2];
            }
            if (t0 + 1 < M) {
                dst[(t0 + 1) * kTile + g] = acc[b][1];
                dst[(t0 + 1) * kTile + g + 8] = acc[b][3];
            }
        }
        __syncwarp();
        mbar_arrive_if(bars + 8u * (kBarSegFull + buf), lane == 0);
        mark(p, ts == 0 ? 5 : 6);
        if (++buf == p.nbuf) {
            buf = 0;
            dphase = dfirst ? 0u : dphase ^ 1u;
            dfirst = false;
        }
    }
    return true;
}

// Epilogue warp of the 16-bit form.  Lane (g, tq) finishes rows g and g + 8 of the tile for the tokens 4cb + tq
// (cb = column block of the up-projection MMA, whose columns 2tq, 2tq + 1 are that token's two 16-bit terms).
// With K slices the tile's partial sums meet in scratch and the slice that arrives last finishes the tile.
template <typename T>
__device__ __forceinline__ bool epilogue_wide(const GemvParams &p, uint8_t *smem, const CUtensorMap *bmap, int lane, int tile_first,
                                              int ntile, int slice)
{
    const int g = lane >> 2, tq = lane & 3;
    const uint32_t sbase = smem_u32(smem), bars = sbase + p.off_bar;
    const uint32_t bring = sbase + p.off_B;
    const int rank = p.rank, M = p.M, nkb = rank / 16, ncb = (M + 3) / 4, SK = p.SK;
    const int nbox = (rank + 63) / 64;
    const uint32_t box_bytes = (uint32_t)kTile * (uint32_t)p.b_box_cols * 2u;
    auto request_b = [&](int ts) {
        const uint32_t bar = bars + 8u * (kBarB + ts % p.nb);
        mbar_expect_tx(bar, (uint32_t)nbox * box_bytes);
        for (int b = 0; b < nbox; ++b)
            tma_load_2d(bring + (uint32_t)(ts % p.nb) * (uint32_t)p.b_slot_bytes + (uint32_t)b * box_bytes, bmap, b * 64,
                        (tile_first + ts) * kTile, bar);
    };
    if (rank > 0 && lane == 0)
        for (int ts = 0; ts < min(ntile, p.nb); ++ts) request_b(ts);   // rows of B are weights: before the wait

    prefetch_x(p, (int)blockIdx.x - p.n_t, lane, (int)sizeof(T));
    uint32_t *s_tf = reinterpret_cast<uint32_t *>(smem + p.off_tf);      // [cb][kb][lane][2]
    for (int i = lane; i < ncb * nkb * 64; i += 32) s_tf[i] = 0u;
    __syncwarp();
    pdl_wait();
    mark(p, 2);

    float isc = 1.f;
    if (rank > 0) {
        float *s_t = reinterpret_cast<float *>(smem + p.off_t);
        float amax = 0.f;
        const size_t slot_elems = (size_t)p.slot_elems;
        const int s_first = p.t_final ? p.n_t : 0, s_end = p.t_final ? p.n_t + 1 : p.n_t;
        bool ok = false;
        for (uint32_t look = 0; look < p.poll_limit && !ok; ++look) {
            bool all = true;
            amax = 0.f;
            if (s_end - s_first > 1) {
                all = look_slots(p.tpart, slot_elems, s_first, s_end, M * rank, lane, s_t, amax);
            } else {
                const uint4 *slot = reinterpret_cast<const uint4 *>(p.tpart + (size_t)s_first * slot_elems);
                for (int q0 = 0; 4 * q0 < M * rank; q0 += 32 * 8) {  // one slot: eight times four entries per lane in flight
                    uint4 part[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const int q = q0 + u * 32 + lane;
                        part[u] = (4 * q < M * rank) ? __ldcg(slot + q) : make_uint4(kTNone, kTNone, kTNone, kTNone);
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const int q = q0 + u * 32 + lane;
                        all = all && t_min(0xFFFFFFFFu, part[u]) != 0u;
                        if (4 * q < M * rank) {
                            const float4 v = make_float4(__uint_as_float(part[u].x), __uint_as_float(part[u].y), __uint_as_float(part[u].z),
                                                         __uint_as_float(part[u].w));
                            *reinterpret_cast<float4 *>(s_t + 4 * q) = v;
                            amax = fmaxf(amax, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
                        }
                    }
                }
            }
            ok = __all_sync(0xffffffffu, all);
            if (!ok && look > 256) __nanosleep(64);
        }
        if (!ok) return false;
        // tell that this CTA has read t (nobody waits for the add; a t CTA clears up once all have told)
        if (lane == 0) atomicAdd(p.ctr + 1, 1);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        __syncwarp();
        const uint32_t ex = min(max(__float_as_uint(amax) >> 23, 1u), 254u);
        const uint32_t sb = min(max(268u - ex, 1u), 254u);
        const float sc = __uint_as_float(sb << 23);
        isc = __uint_as_float((254u - sb) << 23);
        // t as MMA column operands [column block of four tokens][rank block][lane][2]: column 2 (tok % 4) holds the
        // rounded values of token tok, the next column what the rounding left; a lane takes pairs of consecutive rank
        // indices and forms both terms once; the columns of tokens beyond M were set to zero before the wait.
        const int half_rank = rank >> 1;
        for (int idx = lane; idx < M * half_rank; idx += 32) {
            const int tok = idx / half_rank, k0 = 2 * (idx - tok * half_rank);
            const float2 tv = *reinterpret_cast<const float2 *>(s_t + tok * rank + k0);
            const float v0 = tv.x * sc, v1 = tv.y * sc;
            const T h0 = ActTraits<T>::from_float(v0), h1 = ActTraits<T>::from_float(v1);
            const T l0 = ActTraits<T>::from_float(v0 - ActTraits<T>::to_float(h0));
            const T l1 = ActTraits<T>::from_float(v1 - ActTraits<T>::to_float(h1));
            const uint32_t pk_hi = (uint32_t)(*reinterpret_cast<const uint16_t *>(&h0)) | ((uint32_t)(*reinterpret_cast<const uint16_t *>(&h1)) << 16);
            const uint32_t pk_lo = (uint32_t)(*reinterpret_cast<const uint16_t *>(&l0)) | ((uint32_t)(*reinterpret_cast<const uint16_t *>(&l1)) << 16);
            const int cb = tok >> 2, kb = k0 >> 4, h = (k0 >> 3) & 1, q = (k0 & 7) >> 1;
            uint32_t *dst = s_tf + ((size_t)(cb * nkb + kb) * 32 + (2 * (tok & 3)) * 4 + q) * 2 + h;
            dst[0] = pk_hi;
            dst[8] = pk_lo;                                     // four lanes on: the remainder's column
        }
        __syncwarp();
    }
    mark(p, 3);

    const float *s_seg = reinterpret_cast<const float *>(smem + p.off_seg);
    T *y = static_cast<T *>(p.y);
    const uint32_t smask = (uint32_t)p.b_swz, pitch = (uint32_t)p.b_box_cols * 2u;
    const uint32_t tf_lane = sbase + p.off_tf + (uint32_t)lane * 8u;
    // adds t.B^T (rows of B from slot ts % nb) to the sums of a tile and stores its rows of y
    auto finish_tile = [&](int ts, float (&vg)[4], float (&vh)[4]) -> bool {
        const int tile = tile_first + ts;
        if (rank > 0) {
            const int bs = ts % p.nb;
            if (!mbar_wait(bars + 8u * (kBarB + bs), (uint32_t)(ts / p.nb) & 1u)) return false;
            const uint32_t bt = bring + (uint32_t)bs * (uint32_t)p.b_slot_bytes;
            float d[4][4];
#pragma unroll
            for (int cb = 0; cb < 4; ++cb) d[cb][0] = d[cb][1] = d[cb][2] = d[cb][3] = 0.f;
#pragma unroll 1
            for (int kc = 0; 4 * kc < nkb; ++kc) {
                uint32_t af[4][4];
                const uint32_t bx = bt + (uint32_t)kc * box_bytes;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint32_t c0 = (uint32_t)(q * 32 + tq * 4);                  // bytes into the row
                    const uint32_t o0 = (uint32_t)g * pitch + c0, o1 = o0 + 8u * pitch;
                    const bool on = 4 * kc + q < nkb;
                    af[q][0] = on ? lds_u32(bx + swz(o0, smask)) : 0u;
                    af[q][1] = on ? lds_u32(bx + swz(o1, smask)) : 0u;
                    af[q][2] = on ? lds_u32(bx + swz(o0 + 16u, smask)) : 0u;
                    af[q][3] = on ? lds_u32(bx + swz(o1 + 16u, smask)) : 0u;
                }
#pragma unroll
                for (int cb = 0; cb < 4; ++cb) {
                    if (cb < ncb) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            if (4 * kc + q < nkb) {
                                const uint32_t ta = tf_lane + (uint32_t)((cb * nkb + 4 * kc + q) * 32) * 8u;
                                Mma16<T>::run(d[cb], af[q][0], af[q][1], af[q][2], af[q][3], lds_u32(ta), lds_u32(ta + 4u));
                            }
                        }
                    }
                }
            }
#pragma unroll
            for (int cb = 0; cb < 4; ++cb) {
                vg[cb] = fmaf(d[cb][0] + d[cb][1], isc, vg[cb]);
                vh[cb] = fmaf(d[cb][2] + d[cb][3], isc, vh[cb]);
            }
        }
        const int n = tile * kTile + g;
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
            const int tok = 4 * cb + tq;
            if (tok < M) {
                if (n < p.N) y[(size_t)tok * p.N + n] = ActTraits<T>::from_float(vg[cb]);
                if (n + 8 < p.N) y[(size_t)tok * p.N + n + 8] = ActTraits<T>::from_float(vh[cb]);
            }
        }
        return true;
    };
    // B slot of tile ts is free (used or not needed): request the rows of a later tile into it
    auto release_b = [&](int ts) -> bool {
        if (rank == 0) return true;
        // a slice that does not finish the tile never reads its rows of B, but their copy must have landed
        // before the slot is handed out again
        if (!mbar_wait(bars + 8u * (kBarB + ts % p.nb), (uint32_t)(ts / p.nb) & 1u)) return false;
        __syncwarp();
        if (lane == 0 && ts + p.nb < ntile) request_b(ts + p.nb);
        return true;
    };
    // With K slices: whether the tile is ours to finish shows in the arrival count, which is looked at one tile
    // later so that the round trip of its atomic overlaps the next tile's sums.
    int pend_ts = -1, pend_old = 0;
    auto settle = [&](void) -> bool {
        if (pend_ts < 0) return true;
        const int last = __shfl_sync(0xffffffffu, pend_old, 0) == SK - 1;
        if (last) {
            const int tile = tile_first + pend_ts;
            const float *pt = p.part + ((size_t)tile * SK) * M * kTile;
            __threadfence();
            float vg[4], vh[4];
#pragma unroll
            for (int cb = 0; cb < 4; ++cb) {
                const int tok = 4 * cb + tq;
                vg[cb] = vh[cb] = 0.f;
                if (tok < M)
                    for (int s2 = 0; s2 < SK; ++s2) {                   // slices added in order, whoever finishes
                        vg[cb] += __ldcg(pt + ((size_t)s2 * M + tok) * kTile + g);
                        vh[cb] += __ldcg(pt + ((size_t)s2 * M + tok) * kTile + g + 8);
                    }
            }
            if (lane == 0) atomicExch(p.tctr + tile, 0);
            if (!finish_tile(pend_ts, vg, vh)) return false;
        }
        if (!release_b(pend_ts)) return false;
        pend_ts = -1;
        return true;
    };
    for (int ts = 0; ts < ntile; ++ts) {
        const int buf = ts % p.nbuf, tile = tile_first + ts;
        if (!mbar_wait_idle_warp(bars + 8u * (kBarSegFull + buf), (uint32_t)(ts / p.nbuf) & 1u)) return false;
        if (ts == 0) mark(p, 4);
        float vg[4] = {0.f, 0.f, 0.f, 0.f}, vh[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
            const int tok = 4 * cb + tq;
            if (tok < M) {
                const float *src = s_seg + ((size_t)buf * kCW * M + tok) * kTile;
#pragma unroll
                for (int w = 0; w < kCW; ++w) {
                    vg[cb] += src[(size_t)w * M * kTile + g];
                    vh[cb] += src[(size_t)w * M * kTile + g + 8];
                }
            }
        }
        __syncwarp();
        mbar_arrive_if(bars + 8u * (kBarSegFree + buf), lane == 0);
        if (SK > 1) {
            // this slice's partial tile to scratch, then count in
            float *pt = p.part + ((size_t)tile * SK) * M * kTile;
#pragma unroll
            for (int cb = 0; cb < 4; ++cb) {
                const int tok = 4 * cb + tq;
                if (tok < M) {
                    __stcg(pt + ((size_t)slice * M + tok) * kTile + g, vg[cb]);
                    __stcg(pt + ((size_t)slice * M + tok) * kTile + g + 8, vh[cb]);
                }
            }
            __threadfence();
            __syncwarp();
            int old = 0;
            if (lane == 0) old = atomicAdd(p.tctr + tile, 1);
            if (!settle()) return false;                                 // the tile before this one
            pend_ts = ts;
            pend_old = old;
        } else {
            if (!finish_tile(ts, vg, vh)) return false;
            if (!release_b(ts)) return false;
        }
        mark(p, ts == 0 ? 5 : 6);
    }
    if (!settle()) return false;
    return true;
}

// ------------------------------------------------------------------------ t CTA
// Block c of the first n_t: t_kb blocks of 64 input channels of all `rank` rows of A in shared memory
// (TMA, 128-byte swizzle), against the same channels of x read straight from global memory as MMA
// column operands (tokens are columns).  Warps take the 64-channel blocks round-robin (two each at
// most); the eight warps' sums are added in warp order and stored to slot c of tpart.
template <typename T>
__device__ __forceinline__ void t_cta(const GemvParams &p, uint8_t *smem, const CUtensorMap *amap, int c)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tq = lane & 3;
    const uint32_t sbase = smem_u32(smem), bar = sbase + p.off_bar + 8u * kBarA;
    const uint32_t sA = sbase + p.off_tA;
    const int rank = p.rank, M = p.M, nrb = rank / 16;
    const int kb0 = c * p.t_kb, nkb = max(0, min(p.t_kb, (p.K + kTKB - 1) / kTKB - kb0));
    const uint32_t blk_bytes = (uint32_t)rank * 128u;
    if (tid == 0) {
        mbar_init(bar, 1);
        fence_barrier_init();
        if (nkb > 0) {
            mbar_expect_tx(bar, (uint32_t)nkb * blk_bytes);
            for (int b = 0; b < nkb; ++b) tma_load_2d(sA + (uint32_t)b * blk_bytes, amap, (kb0 + b) * kTKB, 0, bar);
        }
    }
    for (int i = tid; i < nkb * M; i += kThreads)      // this CTA's part of x into L2, like the main CTAs' prefetch
        prefetch_l2(static_cast<const T *>(p.x) + (size_t)(i / nkb) * p.K + (size_t)(kb0 + i % nkb) * kTKB);
    __syncthreads();
    mark(p, 1);
    pdl_wait();
    mark(p, 2);
    float *s_red = reinterpret_cast<float *>(smem + p.off_tred);      // [warp][rank][columns in use]
    const int ncol = M <= 2 ? 2 : 8;
    const T *x = static_cast<const T *>(p.x);
    bool dead = false;
    for (int tb = 0; tb < (M + 7) / 8; ++tb) {
        const int tok = tb * 8 + g;
        if (warp < kCW) {
            // this warp's blocks of 64 channels (warp and warp + kCW of the CTA's: two at most): their x as column operands ...
            uint32_t xb[2][4][2];
            bool mine[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                mine[u] = warp + u * kCW < nkb;
                const int k0 = (kb0 + warp + u * kCW) * kTKB;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    const int k = k0 + ks * 16 + 2 * tq;
                    const bool v = mine[u] && tok < M && k < p.K;
                    xb[u][ks][0] = v ? __ldcg(reinterpret_cast<const uint32_t *>(x + (size_t)tok * p.K + k)) : 0u;
                    xb[u][ks][1] = v ? __ldcg(reinterpret_cast<const uint32_t *>(x + (size_t)tok * p.K + k + 8)) : 0u;
                }
            }
            if (mine[0] && !mbar_wait(bar, 0)) dead = true;
            if (tb == 0) mark(p, 3);
            // ... against sixteen rows of A at a time.  Rows are 128 bytes, so the 128-byte swizzle XORs the 16-byte
            // unit index with the row's low three bits, which are this lane's g for all its rows: the swizzled column
            // offsets are constants of the lane.
            const uint32_t xr = (uint32_t)(g & 7) << 4, rowb = (uint32_t)g * 128u;
            uint32_t col[4][2];
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                col[ks][0] = ((uint32_t)(ks * 32 + tq * 4) ^ xr) + rowb;
                col[ks][1] = ((uint32_t)(ks * 32 + tq * 4 + 16) ^ xr) + rowb;
            }
#pragma unroll 1
            for (int r = 0; r < nrb; ++r) {
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    if (mine[u] && !dead) {
                        const uint32_t ab = sA + (uint32_t)(warp + u * kCW) * blk_bytes + (uint32_t)r * 2048u;
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            Mma16<T>::run(acc, lds_u32(ab + col[ks][0]), lds_u32(ab + col[ks][0] + 1024u), lds_u32(ab + col[ks][1]),
                                          lds_u32(ab + col[ks][1] + 1024u), xb[u][ks][0], xb[u][ks][1]);
                    }
                }
                // rows r*16 + g (and + 8) of A, columns 2tq, 2tq+1 (tokens)
                if (2 * tq < ncol) {
                    float *dst = s_red + ((size_t)warp * rank + r * 16 + g) * ncol + 2 * tq;
                    dst[0] = acc[0];
                    dst[1] = acc[1];
                    dst[8 * ncol] = acc[2];
                    dst[8 * ncol + 1] = acc[3];
                }
            }
        }
        __syncthreads();
        const int ntok = min(8, M - tb * 8);
        for (int i = tid; i < ntok * rank; i += kThreads) {
            const int m = i / rank, j = i - m * rank;
            float v = 0.f;
#pragma unroll
            for (int w = 0; w < kCW; ++w) v += s_red[((size_t)w * rank + j) * ncol + m];
            // the value, encoded so that the word is not zero: whoever sees the word sees the value
            p.tpart[(size_t)c * p.slot_elems + (size_t)(tb * 8 + m) * rank + j] = (p.test_skip_arrive || dead) ? 0u : t_enc(v);
        }
        __syncthreads();
    }
    if (dead && lane == 0) give_up(p);
    if (p.t_final) {
        // Many entries (tokens x rank x slots): the t CTA that counts in last adds the slots in order into one
        // more slot, and the main CTAs read that one alone.
        volatile int *s_last = reinterpret_cast<volatile int *>(smem + 512);       // free space between the barriers and A
        __threadfence();
        __syncthreads();
        if (tid == 0) *s_last = (atomicAdd(p.ctr, 1) == p.n_t - 1) ? 1 : 0;
        __syncthreads();
        if (*s_last) {
            __threadfence();
            const size_t slot_elems = (size_t)p.slot_elems;
            if (M * rank <= kThreads) {
                // few entries: one per thread, so that as many threads as possible share the loads
                for (int i = tid; i < M * rank; i += kThreads) {
                    float v = 0.f;
                    bool all = true;
                    for (int c0 = 0; c0 < p.n_t; c0 += 8) {
                        uint32_t part[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) part[u] = (c0 + u < p.n_t) ? __ldcg(p.tpart + (size_t)(c0 + u) * slot_elems + i) : kTNone;
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            v += __uint_as_float(part[u]);
                            all = all && (part[u] != 0u);
                        }
                    }
                    p.tpart[(size_t)p.n_t * slot_elems + i] = all ? t_enc(v) : 0u;
                }
            } else {
                // many entries (several tokens): four per thread and load, or the rounds of loads are this CTA's time
                for (int q = tid; 4 * q < M * rank; q += kThreads) {
                    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                    uint32_t mn = 0xFFFFFFFFu;
                    for (int c0 = 0; c0 < p.n_t; c0 += 8) {
                        uint4 part[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u)
                            part[u] = (c0 + u < p.n_t) ? __ldcg(reinterpret_cast<const uint4 *>(p.tpart + (size_t)(c0 + u) * slot_elems) + q)
                                                       : make_uint4(kTNone, kTNone, kTNone, kTNone);
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            mn = t_min(mn, part[u]);
                            v.x += __uint_as_float(part[u].x);
                            v.y += __uint_as_float(part[u].y);
                            v.z += __uint_as_float(part[u].z);
                            v.w += __uint_as_float(part[u].w);
                        }
                    }
                    reinterpret_cast<uint4 *>(p.tpart + (size_t)p.n_t * slot_elems)[q] =
                        mn != 0u ? make_uint4(t_enc(v.x), t_enc(v.y), t_enc(v.z), t_enc(v.w)) : make_uint4(0u, 0u, 0u, 0u);
                }
            }
        }
    }
    mark(p, 6);
    // Clearing up for the next launch: the readers only tell that they have read t (an add that nobody waits for);
    // one t CTA, which has nothing else left to do, waits until all of them have (bounded), and leaves slots and
    // counters at zero.  That is the CTA that added the slots, or CTA 0 when every reader adds them itself.
    {
        volatile int *s_last = reinterpret_cast<volatile int *>(smem + 512);
        const bool cleaner = p.t_final ? (*s_last != 0) : (c == 0);
        if (cleaner) {
            volatile int *s_ok = s_last + 1;
            if (tid == 0) {
                int ok = 0;
                const unsigned long long t0 = global_ns();
                for (;;) {
                    if (ld_acquire(p.ctr + 1) >= p.n_main) {
                        ok = 1;
                        break;
                    }
                    if (global_ns() - t0 > kWaitNs) break;
                    __nanosleep(100);
                }
                *s_ok = ok;
            }
            __syncthreads();
            if (*s_ok) {
                uint4 *z = reinterpret_cast<uint4 *>(p.tpart);            // 16 bytes per store: this is the kernel's tail
                for (int i = tid; i < (p.n_t + 1) * (p.slot_elems >> 2); i += kThreads) z[i] = make_uint4(0u, 0u, 0u, 0u);
                if (tid == 0) {
                    p.ctr[0] = 0;
                    p.ctr[1] = 0;
                }
            }
        }
    }
}

// ------------------------------------------------------------------------ kernel
template <int BITS, typename T, int M, bool RANKED>
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
gemv_kernel(const GemvParams p, const __grid_constant__ CUtensorMap wmap,
            const __grid_constant__ CUtensorMap bmap, const __grid_constant__ CUtensorMap amap)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);     // the swizzled tiles want 1024-byte alignment
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // the CTAs of the next launch on this stream may become resident as soon as all of ours are
    pdl_launch_dependents();
    mark(p, 0);
    if constexpr (RANKED) {
        if ((int)blockIdx.x < p.n_t) {
            t_cta<T>(p, smem, &amap, (int)blockIdx.x);
            return;
        }
    }
    const int cta = (int)blockIdx.x - p.n_t;
    const int tile_first = (int)((long long)cta * p.NT / p.n_main);
    const int ntile = (int)((long long)(cta + 1) * p.NT / p.n_main) - tile_first;
    const uint32_t bars = smem_u32(smem) + p.off_bar;
    if (tid == 0) {
        prefetch_tensormap(&wmap);
        if (p.rank > 0) prefetch_tensormap(&bmap);
        for (int i = 0; i < p.NS; ++i) {
            mbar_init(bars + 8u * (kBarFull + i), 1);
            mbar_init(bars + 8u * (kBarEmpty + i), kCW);
        }
        for (int i = 0; i < p.nbuf; ++i) {
            mbar_init(bars + 8u * (kBarSegFull + i), kCW);
            mbar_init(bars + 8u * (kBarSegFree + i), 1);
        }
        for (int i = 0; i < p.nb; ++i) mbar_init(bars + 8u * (kBarB + i), 1);
        mbar_init(bars + 8u * kBarXReq, kCW);
        fence_barrier_init();
    }
    __syncthreads();
    mark(p, 1);

    bool ok = true;
    if (warp == kProdWarp) {
        if (lane == 0) ok = produce(p, smem, &wmap, tile_first, ntile);
    } else if (warp == kEpiWarp) {
        ok = epilogue<T, RANKED>(p, smem, &bmap, lane, tile_first, ntile);
    } else {
        pdl_wait();                                  // x may come from the preceding kernel
        mark(p, 2);
        convert_x<BITS, T, M>(p, smem, warp, lane);
        __syncwarp();                                // a warp multiplies only what it has staged itself
        mark(p, 3);
        ok = compute_i8<BITS, T, M>(p, smem, warp, lane, tile_first, ntile);
    }
    if (!ok && lane == 0) give_up(p);
}


// The 16-bit form: main CTA `cta` is row block cta / SK, K slice cta % SK.
template <int BITS, typename T, int MT>
__global__ void __launch_bounds__(kThreads, 1)
gemv_wide_kernel(const GemvParams p, const __grid_constant__ CUtensorMap wmap, const __grid_constant__ CUtensorMap bmap,
                 const __grid_constant__ CUtensorMap amap)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    pdl_launch_dependents();
    mark(p, 0);
    if ((int)blockIdx.x < p.n_t) {
        if (p.pair) cluster_arrive();                // the cluster's barrier counts every thread; nobody here waits on it
        t_cta<T>(p, smem, &amap, (int)blockIdx.x);
        return;
    }
    const int cta = (int)blockIdx.x - p.n_t;
    const int rb = cta / p.SK, slice = cta - rb * p.SK;
    const int tile_first = (int)((long long)rb * p.NT / p.R);
    const int ntile = (int)((long long)(rb + 1) * p.NT / p.R) - tile_first;
    const int g_begin = slice * p.slice_groups, g_count = min(p.slice_groups, p.G - g_begin);
    const uint32_t bars = smem_u32(smem) + p.off_bar;
    if (tid == 0) {
        prefetch_tensormap(&wmap);
        if (p.rank > 0) prefetch_tensormap(&bmap);
        for (int i = 0; i < p.NS; ++i) {
            mbar_init(bars + 8u * (kBarFull + i), 1);
            mbar_init(bars + 8u * (kBarEmpty + i), kCW);
        }
        for (int i = 0; i < p.nbuf; ++i) {
            mbar_init(bars + 8u * (kBarSegFull + i), kCW);
            mbar_init(bars + 8u * (kBarSegFree + i), 1);
        }
        for (int i = 0; i < p.nb; ++i) mbar_init(bars + 8u * (kBarB + i), 1);
        mbar_init(bars + 8u * kBarXReq, kCW);
        fence_barrier_init();
    }
    __syncthreads();
    mark(p, 1);
    bool ok = true;
    if (warp == kProdWarp) {
        if (p.pair) cluster_arrive();
        if (lane == 0) ok = produce(p, smem, &wmap, tile_first, ntile, g_begin, g_count, kCHGW);
    } else if (warp == kEpiWarp) {
        if (p.pair) cluster_arrive();
        ok = epilogue_wide<T>(p, smem, &bmap, lane, tile_first, ntile, slice);
    } else {
        pdl_wait();                                  // x may come from the preceding kernel
        mark(p, 2);
        convert_x16<BITS, T, MT>(p, smem, g_begin, g_count);
        if (p.pair) {                                // both CTAs' halves of x are in both CTAs' shared memory
            cluster_arrive();
            cluster_wait();
        } else {
            named_barrier_sync(1, kCW * 32);
        }
        mark(p, 3);
        ok = compute_w16<BITS, T, MT>(p, smem, warp, lane, ntile, g_begin, g_count);
    }
    if (!ok && lane == 0) give_up(p);
}

// ------------------------------------------------------------------ host side
template <typename X> struct TypeTag { using type = X; };

struct Plan {
    GemvParams p;
    size_t smem;
    bool ok;
};

int g_sm_count = 0;
constexpr size_t kSmemMax = 227 * 1024;

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Fewer t CTAs (two blocks per warp, chunks of A up to 192 KB) where that saves every main CTA a tile: the main
// CTAs are what is left of one CTA per SM, and a launch takes as long as the CTA with the most tiles.
int balanced_t_ctas(int n_t, int nblk, int rank, int tiles, int want)
{
    const int per_max = std::min(2 * kCW, std::max(1, (int)((192 * 1024) / ((size_t)rank * 128))));
    const int n_min = (nblk + per_max - 1) / per_max;
    auto most = [&](int nt) { const int m = std::max(1, std::max(want - nt, want / 2)); return (tiles + m - 1) / m; };
    if (n_min >= n_t || most(n_min) >= most(n_t)) return n_t;
    int best = n_min;
    while (best + 1 < n_t && most(best + 1) == most(n_min)) ++best;
    return best;
}

Plan make_plan(const LinearArgs &a, const GemvTuning &tune)
{
    Plan pl{};
    pl.ok = false;
    if (g_sm_count == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return pl;
        if (cudaDeviceGetAttribute(&g_sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return pl;
    }
    GemvParams &p = pl.p;
    const int GB = (a.bits == 4) ? 64 : 48, G = a.K / kGroupFast;
    p.M = a.M; p.N = a.N; p.K = a.K; p.G = G; p.rank = a.rank;
    p.NT = (a.N + kTile - 1) / kTile;
    const int want = tune.max_ctas > 0 ? tune.max_ctas : g_sm_count;
    const int SPT = (G + kCHG - 1) / kCHG;
    p.stage_bytes = kTile * kCHG * GB;
    p.meta_pitch = (int)align_up((size_t)kTile * G * 2, 16);
    // t CTAs: chunks of A of at most 128 KB (measured at rank 128: 84 us per layer step against 94 with 64 KB chunks)
    p.n_t = 0;
    p.t_kb = 0;
    const int nblk = (a.K + kTKB - 1) / kTKB;
    if (a.rank > 0) {
        const int per = std::min(kCW, std::max(1, (int)((128 * 1024) / ((size_t)a.rank * 128))));     // one block per warp
        p.n_t = std::min(64, std::max((nblk + per - 1) / per, std::min(nblk, 8)));
        p.n_t = balanced_t_ctas(p.n_t, nblk, a.rank, p.NT, want);
        p.t_kb = (nblk + p.n_t - 1) / p.n_t;
        p.n_t = (nblk + p.t_kb - 1) / p.t_kb;
    }
    // All CTAs of a launch, t CTAs included, within one per SM: then every CTA of the NEXT launch finds a free half
    // SM at once.  (Measured: the t CTAs on top of one main CTA per SM cost more, 81 against 72 us per layer step.)
    p.n_main = std::max(1, std::min(std::max(want - p.n_t, want / 2), p.NT));
    const int nseg = (p.NT + p.n_main - 1) / p.n_main;
    p.b_box_cols = a.rank <= 16 ? 16 : (a.rank <= 32 ? 32 : 64);      // columns past the rank arrive as zeros
    p.b_swz = p.b_box_cols >= 64 ? 7 : (p.b_box_cols >= 32 ? 3 : 1);
    p.b_slot_bytes = (int)align_up((size_t)((a.rank + 63) / 64) * kTile * p.b_box_cols * 2, 1024);
    p.nbuf = std::min(kMaxBuf, std::max(2, nseg));
    p.nb = a.rank > 0 ? std::min(kMaxB, std::max(1, nseg)) : 0;
    const int ncol = 3 * a.M;
    auto layout = [&](int ns) {
        p.NS = ns;
        p.nmeta = std::min(kMaxMeta, (ns - 1) / SPT + 2);
        size_t off = 0;
        p.off_bar = (int)off;
        off += (size_t)kNumBars * 8;
        off = align_up(off, 16);
        p.off_tab = (int)off;
        off += (size_t)SPT * kCHG * a.M * 32;                       // the last stage's groups beyond K have (zero) entries too
        off = align_up(off, 128);
        p.off_x = (int)off;
        off += (size_t)G * ncol * (a.bits == 4 ? 128 : 144);
        off = align_up(off, 128);
        p.off_meta = (int)off;
        off += (size_t)p.nmeta * 2 * p.meta_pitch;
        off = align_up(off, 128);
        p.off_seg = (int)off;
        off += (size_t)p.nbuf * kCW * a.M * kTile * 4;
        off = align_up(off, 128);
        p.off_t = (int)off;
        off += (size_t)a.M * a.rank * 4;
        off = align_up(off, 16);
        p.off_tf = (int)off;
        off += (size_t)(a.rank / 16) * 32 * 8;
        p.off_sub = (int)off;
        off += a.rank > 0 ? (size_t)kMaxSub * 32 * 8 : 0;
        off = align_up(off, 1024);
        p.off_B = (int)off;
        off += (size_t)p.nb * p.b_slot_bytes;
        off = align_up(off, 1024);
        p.off_ring = (int)off;
        off += (size_t)ns * p.stage_bytes;
        return off;
    };
    // as many stages as fit the CTA's share of an SM's shared memory (all of a CTA's stages where they are few)
    const size_t budget = (kCtasPerSm == 2 ? 113 * 1024 : kSmemMax) - 2048;
    int ns = std::min(kMaxNS, std::max(2, nseg * SPT));
    while (ns > 2 && layout(ns) > budget) --ns;
    size_t need = layout(ns);
    if (need > budget) {                               // x of a long K: the whole SM
        ns = std::min(kMaxNS, std::max(2, nseg * SPT));
        while (ns > 2 && layout(ns) > kSmemMax - 2048) --ns;
        need = layout(ns);
        if (need > kSmemMax - 2048) return pl;
    }
    // a t CTA: barriers, its blocks of A (1024-byte aligned), the reduction buffer
    p.off_tA = 1024;
    p.off_tred = p.off_tA + p.t_kb * a.rank * 128;
    const size_t need_t = a.rank > 0 ? (size_t)p.off_tred + (size_t)kCW * a.rank * 2 * 4 : 0;      // M <= 2: two columns
    if (need_t > kSmemMax) return pl;
    p.slot_elems = (a.M * a.rank + 31) / 32 * 32;
    p.t_final = (p.n_t * a.M * a.rank > 1024) ? 1 : 0;    // many entries: one t CTA adds the slots for everybody
    pl.smem = std::max(need, need_t) + 1024;       // slack for the alignment of the dynamic window
    p.poll_limit = tune.poll_limit > 0 ? (uint32_t)tune.poll_limit : (1u << 20);
    p.test_skip_arrive = tune.test_skip_arrive;
    pl.ok = true;
    if (getenv("FBQ_PLAN"))
        fprintf(stderr, "gemv plan M %d N %d K %d r %d: n_main %d n_t %d (t_kb %d) NS %d nmeta %d nbuf %d nb %d smem %zu (t CTA %zu)\n",
                a.M, a.N, a.K, a.rank, p.n_main, p.n_t, p.t_kb, p.NS, p.nmeta, p.nbuf, p.nb, need, need_t);
    return pl;
}

// Groups per K slice of the 16-bit form: the smallest power-of-two count of slices whose part of x (16-bit, all
// tokens, whole stages) stays below 136 KB of shared memory.
int wide_slice_groups(int M, int G)
{
    int sk = 1;
    auto slice_of = [&](int k) { return ((G + k - 1) / k + kCHGW - 1) / kCHGW * kCHGW; };
    while (sk < 16 && (size_t)M * ((size_t)slice_of(sk) * kGroupFast + 32) * 2 > 136 * 1024) sk *= 2;
    return slice_of(sk);
}

// Plan of the 16-bit form (3 <= M <= 16): one CTA per SM; K in SK slices when x of all K does not fit.
Plan make_plan_wide(const LinearArgs &a, const GemvTuning &tune)
{
    Plan pl{};
    pl.ok = false;
    if (g_sm_count == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return pl;
        if (cudaDeviceGetAttribute(&g_sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return pl;
    }
    GemvParams &p = pl.p;
    const int GB = (a.bits == 4) ? 64 : 48, G = a.K / kGroupFast, MT = (a.M + 7) / 8;
    p.M = a.M; p.N = a.N; p.K = a.K; p.G = G; p.rank = a.rank;
    p.NT = (a.N + kTile - 1) / kTile;
    const int want = tune.max_ctas > 0 ? tune.max_ctas : g_sm_count;
    p.stage_bytes = kTile * kCHGW * GB;
    p.meta_pitch = (int)align_up((size_t)kTile * G * 2, 16);
    p.n_t = 0;
    p.t_kb = 0;
    const int nblk = (a.K + kTKB - 1) / kTKB;
    if (a.rank > 0) {
        const int per = std::min(kCW, std::max(1, (int)((128 * 1024) / ((size_t)a.rank * 128))));     // one block per warp
        p.n_t = std::min(64, std::max((nblk + per - 1) / per, std::min(nblk, 8)));
        p.n_t = balanced_t_ctas(p.n_t, nblk, a.rank, p.NT, want);
        p.t_kb = (nblk + p.n_t - 1) / p.n_t;
        p.n_t = (nblk + p.t_kb - 1) / p.t_kb;
    }
    // K slices: the smallest power of two whose slice of x (16-bit, all tokens) stays below 136 KB
    p.slice_groups = wide_slice_groups(a.M, G);
    p.SK = (G + p.slice_groups - 1) / p.slice_groups;
    p.x_pitch = p.slice_groups * kGroupFast + 32;
    // One K slice: the main CTAs all stage the same x, so they come in clusters of two that stage half of it each (an
    // even number of t CTAs, the odd one out idle, and of main CTAs keeps the clusters among their own kind).
    p.pair = (p.SK == 1 && p.NT >= 2 && want >= 4) ? 1 : 0;
    if (p.pair && (p.n_t & 1)) ++p.n_t;
    p.R = std::max(1, std::min(std::max(want - p.n_t, want / 2) / p.SK, p.NT));
    if (p.pair && (p.R & 1)) --p.R;
    p.n_main = p.R * p.SK;
    const int nseg = (p.NT + p.R - 1) / p.R;
    // stages per tile of the shortest slice (the last one): the producer runs at most NS stages ahead, that is
    // NS / SPT tiles, and every tile ahead holds a slot of scales and zero points
    const int last_groups = G - (p.SK - 1) * p.slice_groups;
    const int SPT = (std::min(p.slice_groups, last_groups) + kCHGW - 1) / kCHGW;
    p.b_box_cols = a.rank <= 16 ? 16 : (a.rank <= 32 ? 32 : 64);
    p.b_swz = p.b_box_cols >= 64 ? 7 : (p.b_box_cols >= 32 ? 3 : 1);
    p.b_slot_bytes = (int)align_up((size_t)((a.rank + 63) / 64) * kTile * p.b_box_cols * 2, 1024);
    p.nbuf = std::min(kMaxBuf, std::max(2, std::min(nseg, 3)));
    p.nb = a.rank > 0 ? std::min(kMaxB, std::max(1, std::min(nseg, 2))) : 0;
    const int ncb = (a.M + 3) / 4, nkb = a.rank / 16;
    auto layout = [&](int ns) {
        p.NS = ns;
        p.nmeta = std::min(kMaxMeta, (ns - 1) / SPT + 2);
        size_t off = 0;
        p.off_bar = (int)off;
        off += (size_t)kNumBars * 8;
        off = align_up(off, 16);
        p.off_px = (int)off;
        off += (size_t)p.slice_groups * 8 * MT * 8;
        off = align_up(off, 128);
        p.off_x = (int)off;
        off += (size_t)a.M * p.x_pitch * 2;
        off = align_up(off, 128);
        p.off_meta = (int)off;
        off += (size_t)p.nmeta * 2 * p.meta_pitch;
        off = align_up(off, 128);
        p.off_seg = (int)off;
        off += (size_t)p.nbuf * kCW * a.M * kTile * 4;
        off = align_up(off, 128);
        p.off_t = (int)off;
        off += (size_t)a.M * a.rank * 4;
        off = align_up(off, 16);
        p.off_tf = (int)off;
        off += (size_t)ncb * nkb * 32 * 8;
        off = align_up(off, 1024);
        p.off_B = (int)off;
        off += (size_t)p.nb * p.b_slot_bytes;
        off = align_up(off, 1024);
        p.off_ring = (int)off;
        off += (size_t)ns * p.stage_bytes;
        return off;
    };
    int ns = std::min(kMaxNS, (kMaxMeta - 2) * SPT + 1);
    while (ns > 2 && layout(ns) > kSmemMax - 2048) --ns;
    const size_t need = layout(ns);
    if (need > kSmemMax - 2048) return pl;
    p.off_tab = 0;
    p.slot_elems = (a.M * a.rank + 31) / 32 * 32;
    p.t_final = (p.n_t * a.M * a.rank > 2048) ? 1 : 0;
    p.off_tA = 1024;
    p.off_tred = p.off_tA + p.t_kb * a.rank * 128;
    const size_t need_t = a.rank > 0 ? (size_t)p.off_tred + (size_t)kCW * a.rank * 8 * 4 : 0;
    if (need_t > kSmemMax - 2048) return pl;
    pl.smem = std::max(need, need_t) + 1024;
    p.poll_limit = tune.poll_limit > 0 ? (uint32_t)tune.poll_limit : (1u << 20);
    p.test_skip_arrive = tune.test_skip_arrive;
    pl.ok = true;
    if (getenv("FBQ_PLAN"))
        fprintf(stderr, "gemv wide plan M %d N %d K %d r %d: R %d SK %d (slice %d groups) n_t %d NS %d nmeta %d nbuf %d nb %d smem %zu (t CTA %zu)\n",
                a.M, a.N, a.K, a.rank, p.R, p.SK, p.slice_groups, p.n_t, p.NS, p.nmeta, p.nbuf, p.nb, need, need_t);
    return pl;
}

// Tensor maps are encoded on the host once per (pointer, shape) and kept: they hold addresses and
// extents only, never data.
struct MapKey {
    const void *ptr;
    int kind, d0, d1, d2, b0, b1;
    bool operator==(const MapKey &o) const
    {
        return ptr == o.ptr && kind == o.kind && d0 == o.d0 && d1 == o.d1 && d2 == o.d2 && b0 == o.b0 && b1 == o.b1;
    }
};
PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;
std::mutex g_map_mu;
std::vector<std::pair<MapKey, CUtensorMap>> g_maps;
size_t g_map_next = 0;

cudaError_t cached_map(CUtensorMap *out, const MapKey &key, CUtensorMapDataType dt, int ndim, const cuuint64_t *dims,
                       const cuuint64_t *strides, const cuuint32_t *box, CUtensorMapSwizzle swz_mode)
{
    std::lock_guard<std::mutex> lk(g_map_mu);
    for (const auto &e : g_maps)
        if (e.first == key) {
            *out = e.second;
            return cudaSuccess;
        }
    if (!g_encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess) return e;
        if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
        g_encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
    }
    const cuuint32_t estr[3] = {1, 1, 1};
    if (g_encode(out, dt, ndim, const_cast<void *>(key.ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz_mode,
                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    constexpr size_t kKeep = 1024;
    if (g_maps.size() < kKeep)
        g_maps.emplace_back(key, *out);
    else
        g_maps[g_map_next++ % kKeep] = std::make_pair(key, *out);
    return cudaSuccess;
}

template <int BITS, typename T, int MT>
cudaError_t launch_wide(const Plan &pl, const CUtensorMap &wmap, const CUtensorMap &bmap, const CUtensorMap &amap, bool pdl, cudaStream_t s)
{
    auto kern = gemv_wide_kernel<BITS, T, MT>;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemMax);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(pl.p.n_t + pl.p.n_main));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = s;
    cudaLaunchAttribute at[2];
    unsigned na = 0;
    if (pdl) {
        at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    if (pl.p.pair) {
        at[na].id = cudaLaunchAttributeClusterDimension;
        at[na].val.clusterDim.x = 2;
        at[na].val.clusterDim.y = 1;
        at[na].val.clusterDim.z = 1;
        ++na;
    }
    cfg.attrs = at;
    cfg.numAttrs = na;
    return cudaLaunchKernelEx(&cfg, kern, pl.p, wmap, bmap, amap);
}

template <int BITS, typename T, int M, bool RANKED>
cudaError_t launch_variant(const Plan &pl, const CUtensorMap &wmap, const CUtensorMap &bmap, const CUtensorMap &amap, bool pdl,
                           cudaStream_t s)
{
    auto kern = gemv_kernel<BITS, T, M, RANKED>;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemMax);
        if (e != cudaSuccess) return e;
        // Always the largest shared-memory carve-out: launches with different dynamic sizes then share one SM
        // configuration, so the CTAs of consecutive launches can be resident side by side.
        e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(pl.p.n_t + pl.p.n_main));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, pl.p, wmap, bmap, amap);
}

}  // namespace

int gemv_k_slices(int M, int K)
{
    if (M <= 2 || K < kGroupFast) return 1;
    const int G = K / kGroupFast, sg = wide_slice_groups(M, G);
    return (G + sg - 1) / sg;
}

bool gemv_supported(const LinearArgs &a)
{
    if (a.group != kGroupFast || a.K % kGroupFast != 0 || a.K < kGroupFast) return false;
    if (a.M < 1 || a.M > kDecodeMaxM) return false;
    if (a.N % 8 != 0 || a.N < 8) return false;
    if (a.rank % 16 != 0 || a.rank > 128) return false;
    auto mis16 = [](const void *q) { return (reinterpret_cast<uintptr_t>(q) & 15u) != 0; };
    if (mis16(a.scales) || mis16(a.zeros)) return false;
    return true;
}

void gemv_workspace_need(const LinearArgs &a, const GemvTuning &tune, size_t *tpart_floats, int *counters, size_t *partial_floats)
{
    const bool wide = a.M > 2;
    const Plan pl = wide ? make_plan_wide(a, tune) : make_plan(a, tune);
    *tpart_floats = (size_t)(std::max(pl.p.n_t, 1) + 1) * std::max(pl.p.slot_elems, 32);
    *counters = 8 + (wide ? pl.p.NT : 0);
    *partial_floats = (wide && pl.p.SK > 1) ? (size_t)pl.p.NT * pl.p.SK * a.M * kTile : 0;
}

cudaError_t launch_gemv(const LinearArgs &a, Workspace &ws, const GemvTuning &tune, cudaStream_t s, int *launches)
{
    const bool wide = a.M > 2;
    Plan pl = wide ? make_plan_wide(a, tune) : make_plan(a, tune);
    if (!pl.ok) return cudaErrorInvalidConfiguration;
    GemvParams &p = pl.p;
    p.x = a.x; p.scales = a.scales; p.zeros = a.zeros; p.y = a.y;
    p.part = ws.partial;
    p.tctr = ws.counters + 8;
    p.tpart = reinterpret_cast<uint32_t *>(ws.tslots);
    p.ctr = ws.counters;
    p.status = ws.counters + kCtrStatus;
    // tuning aid: consecutive launches write their phase marks to alternate halves of the buffer
    p.trace = nullptr;
    if (ws.trace) {
        static unsigned seq = 0;
        p.trace = reinterpret_cast<unsigned long long *>(ws.trace) + (size_t)(seq++ & 1u) * 256 * kWarps * 16;
        if (p.n_t + p.n_main > 256) p.trace = nullptr;
    }
    CUtensorMap wmap, bmap, amap;
    {
        const cuuint32_t wpg = (a.bits == 4) ? 16 : 12;
        const cuuint64_t dims[3] = {wpg, (cuuint64_t)a.N, (cuuint64_t)p.G};
        const cuuint64_t strides[2] = {(cuuint64_t)p.G * wpg * 4, (cuuint64_t)wpg * 4};
        const int chg = wide ? kCHGW : kCHG;
        const cuuint32_t box[3] = {wpg, (cuuint32_t)kTile, (cuuint32_t)chg};
        const MapKey key{a.qw, 0, (int)wpg, a.N, p.G, kTile, chg};
        if (cudaError_t e = cached_map(&wmap, key, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE);
            e != cudaSuccess)
            return e;
    }
    bmap = wmap;
    amap = wmap;
    if (a.rank > 0) {
        const cuuint64_t bd[2] = {(cuuint64_t)a.rank, (cuuint64_t)a.N}, bs[1] = {(cuuint64_t)a.rank * 2};
        const cuuint32_t bb[2] = {(cuuint32_t)p.b_box_cols, (cuuint32_t)kTile};
        const CUtensorMapSwizzle sw = p.b_swz == 7 ? CU_TENSOR_MAP_SWIZZLE_128B : (p.b_swz == 3 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
        const CUtensorMapDataType dt = a.bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
        if (cudaError_t e = cached_map(&bmap, MapKey{a.B, 1, a.rank, a.N, a.bf16, p.b_box_cols, kTile}, dt, 2, bd, bs, bb, sw); e != cudaSuccess)
            return e;
        const cuuint64_t ad[2] = {(cuuint64_t)a.K, (cuuint64_t)a.rank}, as[1] = {(cuuint64_t)a.K * 2};
        const cuuint32_t ab[2] = {(cuuint32_t)kTKB, (cuuint32_t)a.rank};
        if (cudaError_t e = cached_map(&amap, MapKey{a.A, 2, a.K, a.rank, a.bf16, kTKB, a.rank}, dt, 2, ad, as, ab, CU_TENSOR_MAP_SWIZZLE_128B);
            e != cudaSuccess)
            return e;
    }
    const bool pdl = tune.pdl != 0;
    cudaError_t e = cudaErrorInvalidConfiguration;
    auto go = [&](auto bits, auto type) {
        using T = typename decltype(type)::type;
        constexpr int B = decltype(bits)::value;
        if (a.M > 8) return launch_wide<B, T, 2>(pl, wmap, bmap, amap, pdl, s);
        if (a.M > 2) return launch_wide<B, T, 1>(pl, wmap, bmap, amap, pdl, s);
        if (a.rank == 0)
            return a.M == 1 ? launch_variant<B, T, 1, false>(pl, wmap, bmap, amap, pdl, s) : launch_variant<B, T, 2, false>(pl, wmap, bmap, amap, pdl, s);
        return a.M == 1 ? launch_variant<B, T, 1, true>(pl, wmap, bmap, amap, pdl, s) : launch_variant<B, T, 2, true>(pl, wmap, bmap, amap, pdl, s);
    };
    if (a.bits == 4)
        e = a.bf16 ? go(std::integral_constant<int, 4>{}, TypeTag<__nv_bfloat16>{}) : go(std::integral_constant<int, 4>{}, TypeTag<__half>{});
    else
        e = a.bf16 ? go(std::integral_constant<int, 3>{}, TypeTag<__nv_bfloat16>{}) : go(std::integral_constant<int, 3>{}, TypeTag<__half>{});
    if (e == cudaSuccess) ++*launches;
    return e;
}

}  // namespace fbq
