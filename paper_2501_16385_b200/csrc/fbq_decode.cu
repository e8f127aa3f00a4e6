// Decode kernel (M <= 16) of the FBQuant linear, sm_100a.
//
// One launch computes  y = x.dequant(Q,s,z)^T + (x.A^T).B^T  (Algorithm 1 step 6
// of the paper).  The paper's own kernel (Section 4.3) fuses dequantisation, the
// main product and the up-projection and leaves the down-projection t = x.A^T in
// a second launch; here t is produced by the same launch, so a decode step costs
// one launch per linear and y is written exactly once.
//
// Work split.  The grid is R x SK CTAs: CTA (rr, s) owns the 16-row output tiles
// of row range rr and the quantisation groups of K slice s.  Inside a CTA each
// warp owns whole (tile, slice) tasks.  A task's packed codes are fetched with
// bulk asynchronous copies (one per weight row, mbarrier completion) into a
// small per-warp ring in shared memory, so that every SM keeps tens of KB of
// HBM requests in flight without tying up registers.  Codes are expanded with
// the exponent trick ((w & mask) | 0x6400 is 1024+q in fp16), the zero point is
// subtracted exactly, and the integers q-z are contracted with x by warp-level
// m16n8k16 tensor-core MMAs (16 weight rows x 8 tokens, fp32 accumulation); the
// group scale multiplies the fp32 partial sum once per group.  The k order
// inside an MMA is a fixed permutation chosen so that a lane's packed word IS
// its operand fragment; x is stored in shared memory in the matching order.
//
// Cross-CTA combination is wait-free (no spinning on other CTAs): every task
// writes its fp32 partial tile to scratch and bumps the tile's arrival counter;
// whoever arrives last sums the SK partials in slice order, adds t.B^T and
// stores y.  t is accumulated with fp32 atomics by the warps that own rows of A;
// the warp that completes t publishes a flag and finishes any tile that was
// parked waiting for it.  The only waits in the kernel are on this CTA's own
// bulk copies, and they are bounded.
#include "fbq_common.cuh"

namespace fbq {
namespace {

constexpr int kNW = 8;                 // warps per CTA
constexpr int kThreads = kNW * 32;
constexpr int kTileRows = 16;
constexpr uint32_t kWaitLimit = 1u << 24;

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
    float *partial;     // [SK][M][N]
    float *t;           // [M][rank], zero on entry, zero again on exit
    int *ctr;           // counters, see above; all zero on entry and on exit
    int M, N, K, G, rank;
    int SK, R, NT, CH, D;
    int t_target;       // number of warps that contribute to t
    int t_late;         // test switch: contribute to t after the main loop
    int meta_pitch;     // 8-byte entries per meta row (odd)
    int x_pitch;        // elements per token in shared memory
    int slot_bytes;
    int off_list, off_meta, off_x, off_ring;
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
// Bounded wait: returns false when the limit is hit (never spins forever).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (uint32_t i = 0; i < kWaitLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
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
// unpack(words, z) fills h[0..15] with the pairs (q - z) of one lane's 32 codes
// of one weight row, as packed 16-bit floats, in "fragment order":
//   INT4: h[4i+e]  = codes (8i+e , 8i+e+4)  of word i          (i = 0..3, e = 0..3)
//   INT3: h[5i+f]  = codes (10i+f, 10i+5+f) of word i          (i = 0..2, f = 0..4)
//         h[15]    = codes (30, 31)
// z is the integer zero point of the group.  All arithmetic is exact.
template <int BITS, typename T> struct Unpack;

template <> struct Unpack<4, __half> {
    static constexpr int kWords = 4;
    static __device__ __forceinline__ void run(const uint32_t *w, float z, uint32_t *h)
    {
        const uint32_t c0 = Pk<__half>::splat(1024.f + z), c1 = Pk<__half>::splat(64.f + z);
        const uint32_t sixteenth = 0x2C002C00u;                      // 1/16
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t a = w[i], b = w[i] >> 8;
            h[4 * i + 0] = Pk<__half>::sub(lop3_and_or(a, 0x000F000Fu, 0x64006400u), c0);
            h[4 * i + 1] = Pk<__half>::fma(lop3_and_or(a, 0x00F000F0u, 0x64006400u), sixteenth, c1 ^ 0x80008000u);
            h[4 * i + 2] = Pk<__half>::sub(lop3_and_or(b, 0x000F000Fu, 0x64006400u), c0);
            h[4 * i + 3] = Pk<__half>::fma(lop3_and_or(b, 0x00F000F0u, 0x64006400u), sixteenth, c1 ^ 0x80008000u);
        }
    }
};
template <> struct Unpack<4, __nv_bfloat16> {
    static constexpr int kWords = 4;
    static __device__ __forceinline__ void run(const uint32_t *w, float z, uint32_t *h)
    {
        const uint32_t c0 = Pk<__nv_bfloat16>::splat(128.f + z);     // 0x4300 | q  is 128 + q in bf16
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e)
                h[4 * i + e] = Pk<__nv_bfloat16>::sub(lop3_and_or(w[i] >> (4 * e), 0x000F000Fu, 0x43004300u), c0);
    }
};
template <> struct Unpack<3, __half> {
    static constexpr int kWords = 3;
    static __device__ __forceinline__ void run(const uint32_t *w, float z, uint32_t *h)
    {
        const uint32_t c0 = Pk<__half>::splat(1024.f + z);
        const uint32_t n1 = Pk<__half>::splat(-(128.f + z)), n2 = Pk<__half>::splat(-(16.f + z));
        const uint32_t eighth = 0x30003000u, sixtyfourth = 0x24002400u;   // 1/8, 1/64
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            const uint32_t a = w[i], b = w[i] >> 9;
            h[5 * i + 0] = Pk<__half>::sub(lop3_and_or(a, 0x00070007u, 0x64006400u), c0);
            h[5 * i + 1] = Pk<__half>::fma(lop3_and_or(a, 0x00380038u, 0x64006400u), eighth, n1);
            h[5 * i + 2] = Pk<__half>::fma(lop3_and_or(a, 0x01C001C0u, 0x64006400u), sixtyfourth, n2);
            h[5 * i + 3] = Pk<__half>::sub(lop3_and_or(b, 0x00070007u, 0x64006400u), c0);
            h[5 * i + 4] = Pk<__half>::fma(lop3_and_or(b, 0x00380038u, 0x64006400u), eighth, n1);
        }
        uint32_t l = lop3_and_or(w[0] >> 15, 0x00010001u, 0x64006400u);
        l = lop3_and_or(w[1] >> 14, 0x00020002u, l);
        l = lop3_and_or(w[2] >> 13, 0x00040004u, l);
        h[15] = Pk<__half>::sub(l, c0);
    }
};
template <> struct Unpack<3, __nv_bfloat16> {
    static constexpr int kWords = 3;
    static __device__ __forceinline__ void run(const uint32_t *w, float z, uint32_t *h)
    {
        const uint32_t c0 = Pk<__nv_bfloat16>::splat(128.f + z);
        const uint32_t n1 = Pk<__nv_bfloat16>::splat(-(16.f + z));
        const uint32_t eighth = 0x3E003E00u;                          // 1/8 in bf16
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            const uint32_t a = w[i], b = w[i] >> 6, c = w[i] >> 12;
            h[5 * i + 0] = Pk<__nv_bfloat16>::sub(lop3_and_or(a, 0x00070007u, 0x43004300u), c0);
            h[5 * i + 1] = Pk<__nv_bfloat16>::fma(lop3_and_or(a, 0x00380038u, 0x43004300u), eighth, n1);
            h[5 * i + 2] = Pk<__nv_bfloat16>::sub(lop3_and_or(b, 0x00070007u, 0x43004300u), c0);
            h[5 * i + 3] = Pk<__nv_bfloat16>::fma(lop3_and_or(b, 0x00380038u, 0x43004300u), eighth, n1);
            h[5 * i + 4] = Pk<__nv_bfloat16>::sub(lop3_and_or(c, 0x00070007u, 0x43004300u), c0);
        }
        uint32_t l = lop3_and_or(w[0] >> 15, 0x00010001u, 0x43004300u);
        l = lop3_and_or(w[1] >> 14, 0x00020002u, l);
        l = lop3_and_or(w[2] >> 13, 0x00040004u, l);
        h[15] = Pk<__nv_bfloat16>::sub(l, c0);
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
// Shared-memory element offset of x[k] inside its 128-element group block:
// 16-byte units are laid out [h_index / 4][lane t][h_index % 4] so that one
// 128-bit load per lane fetches the operands of two MMAs, conflict free.
template <int BITS> __device__ __forceinline__ int x_slot(int k_in_group)
{
    const int t = k_in_group >> 5, pos = frag_pos<BITS>(k_in_group & 31);
    const int hidx = pos >> 1;
    return (((hidx >> 2) * 4 + t) * 4 + (hidx & 3)) * 2 + (pos & 1);
}

__device__ __forceinline__ float ld_cg_f32(const float *p) { return __ldcg(p); }
__device__ __forceinline__ int ld_acquire(const int *p)
{
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// --------------------------------------------------------------- tile epilogue
// Sums the SK partial tiles in slice order (or takes `own` when the task was
// not split), adds the up-projection t.B^T and stores y.  Lane (g,t) owns rows
// g and g+8 of the tile and tokens 8b+2t, 8b+2t+1.
template <typename T, int MT>
__device__ __forceinline__ void tile_epilogue(const DecodeParams &p, int tile, int lane, const float (*own)[4])
{
    const int g = lane >> 2, tq = lane & 3;
    const T *B = static_cast<const T *>(p.B);
    T *y = static_cast<T *>(p.y);
#pragma unroll
    for (int b = 0; b < MT; ++b) {
#pragma unroll
        for (int half_row = 0; half_row < 2; ++half_row) {
            const int n = tile * kTileRows + g + 8 * half_row;
#pragma unroll
            for (int tk = 0; tk < 2; ++tk) {
                const int m = 8 * b + 2 * tq + tk;
                if (m >= p.M || n >= p.N) continue;
                float v;
                if (own) {
                    v = own[b][2 * half_row + tk];
                } else {
                    v = 0.f;
                    for (int s = 0; s < p.SK; ++s) v += ld_cg_f32(p.partial + ((size_t)s * p.M + m) * p.N + n);
                }
                if (p.rank > 0) {
                    const uint4 *brow = reinterpret_cast<const uint4 *>(B + (size_t)n * p.rank);
                    const float4 *trow = reinterpret_cast<const float4 *>(p.t + (size_t)m * p.rank);
                    float sub = 0.f;
                    for (int c = 0; c < p.rank / 8; ++c) {
                        const uint4 bv = __ldg(brow + c);
                        const float4 t0 = __ldcg(trow + 2 * c), t1 = __ldcg(trow + 2 * c + 1);
                        const float2 b0 = Pk<T>::to_float2(bv.x), b1 = Pk<T>::to_float2(bv.y);
                        const float2 b2 = Pk<T>::to_float2(bv.z), b3 = Pk<T>::to_float2(bv.w);
                        sub = fmaf(t0.x, b0.x, sub);
                        sub = fmaf(t0.y, b0.y, sub);
                        sub = fmaf(t0.z, b1.x, sub);
                        sub = fmaf(t0.w, b1.y, sub);
                        sub = fmaf(t1.x, b2.x, sub);
                        sub = fmaf(t1.y, b2.y, sub);
                        sub = fmaf(t1.z, b3.x, sub);
                        sub = fmaf(t1.w, b3.y, sub);
                    }
                    v += sub;
                }
                y[(size_t)m * p.N + n] = ActTraits<T>::from_float(v);
            }
        }
    }
}

// Bookkeeping after a tile's y has been stored (and, once per call when there is
// a sub-branch, after the t-completing warp has left its parked-tile loop).
// Whoever retires last restores the scratch invariants (all counters, flags and
// t equal to zero) for the next call on this stream; nobody else is touching the
// scratch space any more at that point.
__device__ __forceinline__ void retire_one(const DecodeParams &p, int lane)
{
    __syncwarp();
    const int target = p.NT + (p.rank > 0 ? 1 : 0);
    int last = 0;
    if (lane == 0) {
        __threadfence();
        last = (atomicAdd(p.ctr + kCtrDone, 1) == target - 1);
    }
    last = __shfl_sync(0xffffffffu, last, 0);
    if (last) {
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

// Claim a parked tile (exactly one claimant wins).
__device__ __forceinline__ bool tile_claim(const DecodeParams &p, int tile, int lane)
{
    int won = 0;
    if (lane == 0) won = (atomicAdd(p.ctr + kCtrFirstTile + tile, 1 << 16) < (1 << 16));
    return __shfl_sync(0xffffffffu, won, 0) != 0;
}

// --------------------------------------------------------------------- kernel
template <int BITS, typename T, int MT>
__global__ void __launch_bounds__(kThreads, 2) decode_kernel(const DecodeParams p)
{
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int GB = (BITS == 4) ? 64 : 48;          // packed bytes of one group of one row
    constexpr int NWORDS = Unpack<BITS, T>::kWords;    // words per lane per group

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, tq = lane & 3;
    const int s = blockIdx.x % p.SK, rr = blockIdx.x / p.SK;
    const int g0 = (int)((long long)s * p.G / p.SK), g1 = (int)((long long)(s + 1) * p.G / p.SK);
    const int ngs = g1 - g0;
    const int tile0 = (int)((long long)rr * p.NT / p.R), tile1 = (int)((long long)(rr + 1) * p.NT / p.R);
    const int ntiles = tile1 - tile0;
    const int nchunks = (ngs + p.CH - 1) / p.CH;
    const int my_tiles = (ntiles > warp) ? (ntiles - warp + kNW - 1) / kNW : 0;
    const int n_items = my_tiles * nchunks;
    const size_t row_bytes = (size_t)p.G * GB;

    uint64_t *bars = reinterpret_cast<uint64_t *>(smem);
    uint2 *s_meta = reinterpret_cast<uint2 *>(smem + p.off_meta);
    T *s_x = reinterpret_cast<T *>(smem + p.off_x);
    const uint32_t ring_base = smem_u32(smem + p.off_ring) + (uint32_t)(warp * p.D) * p.slot_bytes;
    const uint8_t *ring_ptr = smem + p.off_ring + (size_t)(warp * p.D) * p.slot_bytes;
    const uint32_t bar_base = smem_u32(bars + warp * p.D);

    if (tid == 0) {
        for (int i = 0; i < kNW * p.D; ++i) mbar_init(smem_u32(bars + i), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // ---- producer side of this warp's ring ---------------------------------
    auto issue = [&](int it) {
        const int tile = tile0 + warp + (it / nchunks) * kNW;
        const int cg0 = g0 + (it % nchunks) * p.CH;
        const int ng = min(p.CH, g1 - cg0);
        const int slot = it % p.D;
        const uint32_t bar = bar_base + 8u * slot;
        const uint32_t bytes_row = (uint32_t)ng * GB;
        if (lane == 0) mbar_expect_tx(bar, bytes_row * kTileRows);
        __syncwarp();
        if (lane < kTileRows) {
            const int n = min(tile * kTileRows + lane, p.N - 1);
            bulk_g2s(ring_base + slot * p.slot_bytes + lane * bytes_row, p.qw + (size_t)n * row_bytes + (size_t)cg0 * GB,
                     bytes_row, bar);
        }
    };
    for (int it = 0; it < min(p.D, n_items); ++it) issue(it);

    // Everything above touches only the weights, which no earlier kernel of the
    // stream writes; from here on x may come from the previous kernel.
    pdl_wait();
    pdl_launch_dependents();

    // ---- which warps own rows of A (down-projection share) ------------------
    const int j0 = (int)((long long)rr * p.rank / p.R), j1 = (int)((long long)(rr + 1) * p.rank / p.R);
    const int nj = j1 - j0;
    const int ntw = min(nj, kNW);                      // t-warps are the LAST ntw warps
    const bool is_tw = warp >= kNW - ntw;
    const int nfill_warps = (ntw < kNW && !p.t_late) ? kNW - ntw : kNW;   // warps that fill shared memory

    auto t_share = [&]() {
        // t[m][j] += sum_{k in slice} x[m][k] * A[j][k] for this warp's rows j
        const T *A = static_cast<const T *>(p.A);
        const T *x = static_cast<const T *>(p.x);
        const int k0 = g0 * kGroupFast, k1 = g1 * kGroupFast;
        for (int j = j0 + (kNW - 1 - warp); j < j1; j += ntw) {
            float acc[MT * 8];
#pragma unroll
            for (int m = 0; m < MT * 8; ++m) acc[m] = 0.f;
            for (int k = k0 + lane * 8; k < k1; k += 256) {
                const uint4 av = __ldg(reinterpret_cast<const uint4 *>(A + (size_t)j * p.K + k));
                const float2 a0 = Pk<T>::to_float2(av.x), a1 = Pk<T>::to_float2(av.y);
                const float2 a2 = Pk<T>::to_float2(av.z), a3 = Pk<T>::to_float2(av.w);
#pragma unroll
                for (int m = 0; m < MT * 8; ++m) {
                    if (m < p.M) {
                        const uint4 xv = __ldcg(reinterpret_cast<const uint4 *>(x + (size_t)m * p.K + k));
                        const float2 x0 = Pk<T>::to_float2(xv.x), x1 = Pk<T>::to_float2(xv.y);
                        const float2 x2 = Pk<T>::to_float2(xv.z), x3 = Pk<T>::to_float2(xv.w);
                        float v = acc[m];
                        v = fmaf(x0.x, a0.x, v);
                        v = fmaf(x0.y, a0.y, v);
                        v = fmaf(x1.x, a1.x, v);
                        v = fmaf(x1.y, a1.y, v);
                        v = fmaf(x2.x, a2.x, v);
                        v = fmaf(x2.y, a2.y, v);
                        v = fmaf(x3.x, a3.x, v);
                        v = fmaf(x3.y, a3.y, v);
                        acc[m] = v;
                    }
                }
            }
#pragma unroll
            for (int m = 0; m < MT * 8; ++m) {
                if (m < p.M) {
                    float v = acc[m];
                    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                    if (lane == 0) atomicAdd(p.t + (size_t)m * p.rank + j, v);
                }
            }
        }
    };
    // After this warp's share of t is in: count it; the warp that completes t
    // publishes the flag and finishes every tile parked before the flag was up.
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
        for (int i = 0; i < npend; ++i) {
            int tile = 0;
            if (lane == 0) tile = ld_acquire(p.ctr + kCtrFirstTile + p.NT + i) - 1;
            tile = __shfl_sync(0xffffffffu, tile, 0);
            if (tile < 0) continue;                    // entry not visible yet: its owner will see the flag
            if (!tile_claim(p, tile, lane)) continue;
            __threadfence();
            tile_epilogue<T, MT>(p, tile, lane, nullptr);
            retire_one(p, lane);
        }
        retire_one(p, lane);                           // the completer's own slot in the retire count
    };

    if (p.rank > 0 && is_tw && !p.t_late) t_share();

    // ---- fill shared memory: permuted x slice and (scale, zero) table --------
    if (warp < nfill_warps) {
        const int nthr = nfill_warps * 32;
        const T *x = static_cast<const T *>(p.x);
        const int kslice = ngs * kGroupFast;
        for (int idx = tid; idx < p.M * (kslice / 8); idx += nthr) {
            const int m = idx / (kslice / 8), kk = (idx - m * (kslice / 8)) * 8;
            const uint4 v = __ldcg(reinterpret_cast<const uint4 *>(x + (size_t)m * p.K + g0 * kGroupFast + kk));
            const uint16_t *e = reinterpret_cast<const uint16_t *>(&v);
            uint16_t *dst = reinterpret_cast<uint16_t *>(s_x + (size_t)m * p.x_pitch + (kk >> 7) * kGroupFast);
#pragma unroll
            for (int i = 0; i < 8; ++i) dst[x_slot<BITS>((kk & 127) + i)] = e[i];
        }
        const int nrows = ntiles * kTileRows;
        for (int idx = tid; idx < nrows * ngs; idx += nthr) {
            const int r = idx / ngs, gl = idx - r * ngs;
            const int n = min(tile0 * kTileRows + r, p.N - 1);
            const float sc = __half2float(p.scales[(size_t)n * p.G + g0 + gl]);
            const float ze = __half2float(p.zeros[(size_t)n * p.G + g0 + gl]);
            s_meta[(size_t)r * p.meta_pitch + gl] = make_uint2(__float_as_uint(sc), __float_as_uint(ze));
        }
    }
    __syncthreads();
    if (p.rank > 0 && is_tw && !p.t_late) t_arrive();

    // ---- consumer: stream this warp's tasks ---------------------------------
    bool dead = false;
    int it = 0;
    for (int ti = 0; ti < my_tiles && !dead; ++ti) {
        const int tile = tile0 + warp + ti * kNW;
        float acc[MT][4];
#pragma unroll
        for (int b = 0; b < MT; ++b)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[b][i] = 0.f;

        for (int ch = 0; ch < nchunks; ++ch, ++it) {
            const int slot = it % p.D;
            if (!mbar_wait(bar_base + 8u * slot, (uint32_t)(it / p.D) & 1u)) {
                dead = true;
                break;
            }
            const int cgl = ch * p.CH;                          // first group of the chunk, slice-local
            const int ng = min(p.CH, ngs - cgl);
            const uint8_t *slot_ptr = ring_ptr + (size_t)slot * p.slot_bytes;
            const uint32_t bytes_row = (uint32_t)ng * GB;
            const uint2 *meta_a = s_meta + (size_t)((tile - tile0) * kTileRows + g) * p.meta_pitch + cgl;
            const uint2 *meta_b = meta_a + (size_t)8 * p.meta_pitch;

            for (int gi = 0; gi < ng; ++gi) {
                const uint2 ma = meta_a[gi], mb = meta_b[gi];
                uint32_t wa[NWORDS], wb[NWORDS];
                const uint8_t *pa = slot_ptr + (size_t)g * bytes_row + gi * GB + tq * (GB / 4);
                const uint8_t *pb = pa + (size_t)8 * bytes_row;
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
                Unpack<BITS, T>::run(wa, __uint_as_float(ma.y), ha);
                Unpack<BITS, T>::run(wb, __uint_as_float(mb.y), hb);

                float tmp[MT][4];
#pragma unroll
                for (int b = 0; b < MT; ++b) {
                    tmp[b][0] = tmp[b][1] = tmp[b][2] = tmp[b][3] = 0.f;
                    const int token = 8 * b + g;
                    const uint4 *xg = reinterpret_cast<const uint4 *>(s_x + (size_t)token * p.x_pitch +
                                                                      (size_t)(cgl + gi) * kGroupFast);
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint4 xv = make_uint4(0u, 0u, 0u, 0u);
                        if (token < p.M) xv = xg[q4 * 4 + tq];
                        const uint32_t a0[4] = {ha[4 * q4 + 0], hb[4 * q4 + 0], ha[4 * q4 + 1], hb[4 * q4 + 1]};
                        const uint32_t a1[4] = {ha[4 * q4 + 2], hb[4 * q4 + 2], ha[4 * q4 + 3], hb[4 * q4 + 3]};
                        Pk<T>::mma(tmp[b], a0, xv.x, xv.y);
                        Pk<T>::mma(tmp[b], a1, xv.z, xv.w);
                    }
                    const float sa = __uint_as_float(ma.x), sb = __uint_as_float(mb.x);
                    acc[b][0] = fmaf(sa, tmp[b][0], acc[b][0]);
                    acc[b][1] = fmaf(sa, tmp[b][1], acc[b][1]);
                    acc[b][2] = fmaf(sb, tmp[b][2], acc[b][2]);
                    acc[b][3] = fmaf(sb, tmp[b][3], acc[b][3]);
                }
            }
            // slot consumed: refill it with the task D items ahead
            __syncwarp();
            if (it + p.D < n_items) {
                fence_proxy_async();
                issue(it + p.D);
            }
        }
        if (dead) break;

        // ---- hand the finished (tile, slice) task over ------------------------
        if (p.SK == 1 && p.rank == 0) {
            tile_epilogue<T, MT>(p, tile, lane, acc);
            continue;
        }
#pragma unroll
        for (int b = 0; b < MT; ++b)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int n = tile * kTileRows + g + 8 * (i >> 1), m = 8 * b + 2 * tq + (i & 1);
                if (m < p.M && n < p.N) p.partial[((size_t)s * p.M + m) * p.N + n] = acc[b][i];
            }
        __syncwarp();
        int last = 0;
        if (lane == 0) {
            __threadfence();
            last = ((atomicAdd(p.ctr + kCtrFirstTile + tile, 1) & 0xFFFF) == p.SK - 1);
        }
        last = __shfl_sync(0xffffffffu, last, 0);
        if (!last) continue;
        if (p.rank > 0) {
            int ready = 0;
            if (lane == 0) {
                __threadfence();
                ready = ld_acquire(p.ctr + kCtrReady);
                if (!ready) {
                    // park the tile, then look again: either we see the flag now, or the
                    // warp that raises it will see our entry (both sides fence in between)
                    const int idx = atomicAdd(p.ctr + kCtrPendingN, 1);
                    atomicExch(p.ctr + kCtrFirstTile + p.NT + idx, tile + 1);
                    __threadfence();
                    ready = ld_acquire(p.ctr + kCtrReady) ? 2 : 0;
                }
            }
            ready = __shfl_sync(0xffffffffu, ready, 0);
            if (ready == 0) continue;                               // parked: finished by the t-completing warp
            if (ready == 2 && !tile_claim(p, tile, lane)) continue; // parked and already taken
        }
        __threadfence();
        tile_epilogue<T, MT>(p, tile, lane, nullptr);
        retire_one(p, lane);
    }

    if (dead) {
        // A bulk copy did not complete in time: report, give copies already in flight a
        // last bounded chance to land (the CTA must not exit under them), and stop.
        if (lane == 0) atomicExch(p.ctr + kCtrStatus, (int)FBQ_ERR_TIMEOUT);
        for (int j = it; j < min(it + p.D, n_items); ++j)
            (void)mbar_wait(bar_base + 8u * (j % p.D), (uint32_t)(j / p.D) & 1u);
    }
    if (p.rank > 0 && is_tw && p.t_late) {
        t_share();
        t_arrive();
    }
}

// ------------------------------------------------------------------ host side
struct Plan {
    int SK, R, NT, CH, D, t_target;
    int meta_pitch, x_pitch, slot_bytes;
    int off_list, off_meta, off_x, off_ring;
    size_t smem;
    bool ok;
};

int g_sm_count = 0;

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
    pl.NT = (a.N + kTileRows - 1) / kTileRows;
    int max_ctas = 2 * g_sm_count;
    if (tune.max_ctas > 0) max_ctas = min(max_ctas, tune.max_ctas);
    // K slices: enough (tile, slice) tasks to give every warp of the grid about
    // two, but never more slices than groups, and fewer for many tokens (each
    // slice costs one fp32 partial tile per output tile).
    int sk = tune.sk;
    if (sk <= 0) {
        const long long want_tasks = 2LL * max_ctas * kNW;
        sk = (int)((want_tasks + pl.NT - 1) / pl.NT);
        const int cap = (a.M <= 2) ? 16 : (a.M <= 8 ? 8 : 4);
        sk = max(1, min(sk, cap));
    }
    sk = max(1, min(sk, G));
    pl.SK = sk;
    pl.R = max(1, min(max_ctas / sk, pl.NT));
    const int ngs_max = (G + sk - 1) / sk;
    pl.CH = tune.chunk > 0 ? tune.chunk : 3;
    pl.CH = max(1, min(pl.CH, ngs_max));
    pl.D = tune.depth > 0 ? tune.depth : 2;
    pl.slot_bytes = kTileRows * pl.CH * GB;
    const int tiles_max = (pl.NT + pl.R - 1) / pl.R;
    pl.meta_pitch = ngs_max | 1;
    pl.x_pitch = ngs_max * kGroupFast + 32;    // +64 bytes: tokens 2j, 2j+1 land in different bank halves
    size_t off = (size_t)kNW * pl.D * 8;
    pl.off_list = (int)off;
    off = (off + 15) & ~(size_t)15;
    pl.off_meta = (int)off;
    off += (size_t)tiles_max * kTileRows * pl.meta_pitch * 8;
    off = (off + 127) & ~(size_t)127;
    pl.off_x = (int)off;
    off += (size_t)a.M * pl.x_pitch * 2;
    off = (off + 127) & ~(size_t)127;
    pl.off_ring = (int)off;
    off += (size_t)kNW * pl.D * pl.slot_bytes;
    pl.smem = off;
    // warps that own at least one row of A
    pl.t_target = 0;
    if (a.rank > 0) {
        for (int rr = 0; rr < pl.R; ++rr) {
            const int nj = (int)((long long)(rr + 1) * a.rank / pl.R) - (int)((long long)rr * a.rank / pl.R);
            pl.t_target += min(nj, kNW);
        }
        pl.t_target *= pl.SK;
    }
    pl.ok = pl.smem <= 110 * 1024;
    return pl;
}

template <int BITS, typename T, int MT>
cudaError_t launch_variant(const DecodeParams &p, const Plan &pl, bool pdl, cudaStream_t s)
{
    auto kern = decode_kernel<BITS, T, MT>;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 112 * 1024);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(pl.R * pl.SK));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, p);
}

int g_t_late = 0;

}  // namespace

void decode_set_test_switch(int t_late) { g_t_late = t_late; }

void decode_workspace_need(const LinearArgs &a, const DecodeTuning &tune, size_t *partial_floats, int *counters)
{
    const Plan pl = make_plan(a, tune);
    *partial_floats = (size_t)pl.SK * a.M * a.N;
    *counters = kCtrFirstTile + 2 * pl.NT;
}

cudaError_t launch_decode(const LinearArgs &a, Workspace &ws, const DecodeTuning &tune, cudaStream_t s, int *launches)
{
    const Plan pl = make_plan(a, tune);
    if (!pl.ok) return cudaErrorInvalidConfiguration;
    DecodeParams p{};
    p.x = a.x;
    p.qw = reinterpret_cast<const uint8_t *>(a.qw);
    p.scales = a.scales;
    p.zeros = a.zeros;
    p.A = a.A;
    p.B = a.B;
    p.y = a.y;
    p.partial = ws.partial;
    p.t = ws.t;
    p.ctr = ws.counters;
    p.M = a.M; p.N = a.N; p.K = a.K; p.G = a.K / kGroupFast; p.rank = a.rank;
    p.SK = pl.SK; p.R = pl.R; p.NT = pl.NT; p.CH = pl.CH; p.D = pl.D;
    p.t_target = pl.t_target;
    p.t_late = g_t_late;
    p.meta_pitch = pl.meta_pitch; p.x_pitch = pl.x_pitch; p.slot_bytes = pl.slot_bytes;
    p.off_list = pl.off_list; p.off_meta = pl.off_meta; p.off_x = pl.off_x; p.off_ring = pl.off_ring;
    const bool pdl = tune.pdl != 0;
    cudaError_t e;
    const int mt = (a.M <= 8) ? 1 : 2;
    if (a.bf16) {
        if (a.bits == 4) e = (mt == 1) ? launch_variant<4, __nv_bfloat16, 1>(p, pl, pdl, s) : launch_variant<4, __nv_bfloat16, 2>(p, pl, pdl, s);
        else             e = (mt == 1) ? launch_variant<3, __nv_bfloat16, 1>(p, pl, pdl, s) : launch_variant<3, __nv_bfloat16, 2>(p, pl, pdl, s);
    } else {
        if (a.bits == 4) e = (mt == 1) ? launch_variant<4, __half, 1>(p, pl, pdl, s) : launch_variant<4, __half, 2>(p, pl, pdl, s);
        else             e = (mt == 1) ? launch_variant<3, __half, 1>(p, pl, pdl, s) : launch_variant<3, __half, 2>(p, pl, pdl, s);
    }
    if (e == cudaSuccess) ++*launches;
    return e;
}

}  // namespace fbq
