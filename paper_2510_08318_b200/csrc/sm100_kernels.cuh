// Tensor-core kernels (tcgen05 + TMEM + TMA) for linear attention with the Hedgehog feature map,
// bf16 storage, head dimension 128.  The forward has three steps, run either as ONE persistent
// cooperative kernel (linattn_fused_tc: key side, per-head meeting point, combine, per-head meeting point,
// query side) or as three launches:
//
//   kside_tc   : persistent CTAs stream 128-token tiles of K and V.  Per tile
//                  U = K W_k          (tcgen05.mma, 128x64x128, fp32 in TMEM)                 Eq. 6
//                  phi(k) = softmax(U) (+) softmax(-U)   (CUDA cores, one token per thread; bf16, written
//                                                         over the K tile in shared memory)   Eq. 6
//                  S += phi(k)^T V ,  z += phi(k)^T 1     (tcgen05.mma, accumulators stay in TMEM) Eq. 5
//                one partial (S, z) per (CTA, head) is written to the workspace.
//   combine_tc : fixed-order sum of the partials of each head; emits S as a bf16 image for TMA and z as
//                a bf16 hi+lo pair laid out as a tcgen05 operand.
//   qside_tc   : persistent CTAs stream 128-token tiles of Q.  Per tile
//                  U = Q W_q, phi(q) as above (written over the Q tile)                        Eq. 6
//                  num = phi(q) S ,  den = phi(q) . z      (tcgen05.mma)                      Eq. 5
//                  o = num / den -> bf16, written over the same tile, TMA store                Eq. 5
//
// Work split: the G * ceil(n/128) tiles form one sequence (head-major); CTA c of P owns the contiguous
// run [c*T/P, (c+1)*T/P).  A run may cross head boundaries; each (CTA, head) piece is a "segment".
// Warp roles (16 warps): warps 0-3 feature map softmax(+U), warps 4-7 softmax(-U) (one token per thread),
// warp 8 TMA producer, warp 9 issues the logits MMAs, warp 10 issues the accumulation MMAs, warp 11 issues
// the TMA stores (query side), warps 12-15 query-side epilogue (num / den -> bf16 output tile) and, in the
// fused kernel, every warp but 8 and 9 takes part in the meeting points and the combine step between the two sides.  Role loops are
// warp-uniform; single-thread work (TMA and MMA issue) is predicated inside them.
// Every wait is bounded: on time-out the kernel records a code in *err, raises the CTA's abort word so
// that the other roles stop waiting too, and unwinds.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sm100_ptx.cuh"

namespace linattn {
namespace tc {

using namespace ptx;

constexpr int kD = 128;             // head dimension
constexpr int kM = 64;              // features per softmax half
constexpr int kTile = 128;          // tokens per tile
constexpr int kE = kD * kD + kD;    // floats per (S, z) record
constexpr uint32_t kTileBytes = kTile * kD * 2;       // 32 KB: one [128 x 128] bf16 tile
constexpr uint32_t kHalfTileBytes = kTileBytes / 2;   // one 64-column block of a tile
constexpr uint32_t kWBytes = kM * kD * 2;             // 16 KB: W^T [64 x 128] bf16
constexpr uint32_t kZBlkBytes = 2 * 16 * 128;         // 4 KB: z operand, [2 blocks][16 rows][64] bf16
constexpr uint32_t kWaitLimitUs = 2000u * 1000u;   // default bound of every device-side wait: 2 s
constexpr float kLog2e = 1.4426950408889634f;

// error codes OR-ed into *err (which wait gave up)
enum : uint32_t {
    kErrProducer = 1u, kErrMmaLoad = 2u, kErrMmaU = 4u, kErrMmaPhi = 8u, kErrMmaAcc = 16u,
    kErrSoftmaxU = 32u, kErrDrain = 64u, kErrEpilogue = 128u, kErrSeg = 256u, kErrStore = 512u, kErrGrid = 1024u,
    kErrSmem = 2048u   // not a wait: the kernel's shared-memory window did not hold its layout
};

// CTA that owns tile t when T tiles are split over P CTAs (CTA c owns [c*T/P, (c+1)*T/P)).
__host__ __device__ __forceinline__ long long tile_owner(long long t, long long T, long long P)
{
    return ((t + 1) * P - 1) / T;
}

// Walks this CTA's run of tiles.  g = (batch, head) index, lt = tile within the head, seg = number of
// head boundaries crossed so far; first / last mark the ends of a segment.
struct TileWalk {
    int count, i, g, lt, seg, tiles_per_head;
    __device__ __forceinline__ void init(long long total_tiles, int tph)
    {
        const long long P = gridDim.x, c = blockIdx.x;
        const long long a = c * total_tiles / P, b = (c + 1) * total_tiles / P;
        count = (int)(b - a);
        tiles_per_head = tph;
        g = (int)(a / tph);
        lt = (int)(a % tph);
        i = 0;
        seg = 0;
    }
    __device__ __forceinline__ bool done() const { return i >= count; }
    __device__ __forceinline__ bool first() const { return i == 0 || lt == 0; }
    __device__ __forceinline__ bool last() const { return i == count - 1 || lt == tiles_per_head - 1; }
    __device__ __forceinline__ void next()
    {
        ++i;
        if (++lt == tiles_per_head) {
            lt = 0;
            ++g;
            ++seg;
        }
    }
};

// Ring position: slot index and the parity of the phase a consumer waits for on its n-th visit.
template <int N> struct Ring {
    int s = 0;
    uint32_t ph = 0;
    __device__ __forceinline__ void next()
    {
        if (++s == N) {
            s = 0;
            ph ^= 1u;
        }
    }
};

// What every role needs to wait on a barrier and to report a failed wait.
struct WaitCtx {
    uint32_t* err;        // global error word
    uint32_t abort_smem;  // shared-memory address of the CTA's abort word
    uint32_t limit_us = kWaitLimitUs;   // bound of each wait
    __device__ __forceinline__ uint64_t limit_ns() const { return (uint64_t)limit_us * 1000u; }
};

// All lanes wait (bounded); the verdict is made warp-uniform so that role loops never diverge.
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, const WaitCtx& wc, uint32_t code)
{
    const bool ok = mbar_wait_abortable(bar, parity, wc.limit_ns(), wc.abort_smem);
    const bool all = __all_sync(0xffffffffu, ok);
    if (!all && (threadIdx.x & 31) == 0) {
        atomicOr(wc.err, code);
        asm volatile("st.volatile.shared.u32 [%0], %1;" ::"r"(wc.abort_smem), "r"(1u) : "memory");
    }
    return all;
}

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// ---- packed fp32 pairs (one instruction for two lanes of arithmetic) ----------------------------------
using f32x2 = uint64_t;
__device__ __forceinline__ f32x2 pack2(float lo, float hi)
{
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c)
{
    f32x2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b)
{
    f32x2 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b)
{
    f32x2 r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ float max3(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
__device__ __forceinline__ float min3(float a, float b, float c)
{
    float r;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// 2^x for a pair of x <= 0 on the FMA pipe (no special-function unit): x = i + f with i = round(x),
// f in [-1/2, 1/2]; 2^f by a cubic (relative error < 7.5e-5, far below the bf16 rounding applied to the
// result), then i is added into the exponent field.  x is clamped at -126 (result ~1e-38).
__device__ __forceinline__ f32x2 exp2_poly2(f32x2 x)
{
    float x0, x1;
    unpack2(x, x0, x1);
    x = pack2(fmaxf(x0, -126.f), fmaxf(x1, -126.f));
    const float magic = 12582912.f;  // 1.5 * 2^23: adding it leaves round(x) in the low mantissa bits
    const f32x2 t = add2(x, pack2(magic, magic));
    const f32x2 fi = add2(t, pack2(-magic, -magic));
    const f32x2 f = fma2(fi, pack2(-1.f, -1.f), x);
    f32x2 p = fma2(f, pack2(0.055171459913253784f, 0.055171459913253784f), pack2(0.2426108568906784f, 0.2426108568906784f));
    p = fma2(p, f, pack2(0.6932609677314758f, 0.6932609677314758f));
    p = fma2(p, f, pack2(0.9999281167984009f, 0.9999281167984009f));
    float p0, p1, t0, t1;
    unpack2(p, p0, p1);
    unpack2(t, t0, t1);
    const float r0 = __uint_as_float(__float_as_uint(p0) + (__float_as_uint(t0) << 23));
    const float r1 = __uint_as_float(__float_as_uint(p1) + (__float_as_uint(t1) << 23));
    return pack2(r0, r1);
}

// One softmax half of Eq. 6 for one token.  u[64] holds the logits of this thread's token on entry.
// kNeg = false: softmax(+u); kNeg = true: softmax(-u).  The 64 results, scaled by `keep` (0 for rows
// past the end of the sequence), are written as bf16 to `row_base` = start of this token's 128-byte row
// in the 64-feature block, 16-byte chunk c stored at chunk c ^ (row & 7) (the 128-byte swizzle).
// Arithmetic is fp32, two lanes per instruction; one pair in four takes its exponentials on the FMA
// pipe (exp2_poly2) so that the special-function unit and the FMA pipe finish together.
template <bool kNeg>
__device__ __forceinline__ void softmax_half_to_smem(float (&u)[kM], float keep, uint8_t* row_base, int row)
{
    float m = kNeg ? min3(u[0], u[1], u[2]) : max3(u[0], u[1], u[2]);
#pragma unroll
    for (int j = 3; j < kM - 1; j += 2) m = kNeg ? min3(m, u[j], u[j + 1]) : max3(m, u[j], u[j + 1]);
    m = kNeg ? fminf(m, u[kM - 1]) : fmaxf(m, u[kM - 1]);
    // exp(u - max) = 2^(u*log2e - max*log2e);   exp(-u - max(-u)) = 2^(min*log2e - u*log2e)
    const float sL = kNeg ? -kLog2e : kLog2e;
    const float off = kNeg ? m * kLog2e : -m * kLog2e;
    const f32x2 scale = pack2(sL, sL), offset = pack2(off, off);
    f32x2 e[kM / 2];
    f32x2 sum2 = pack2(0.f, 0.f);
#pragma unroll
    for (int p = 0; p < kM / 2; ++p) {
        const f32x2 x = fma2(pack2(u[2 * p], u[2 * p + 1]), scale, offset);
        if ((p & 3) == 3) {
            e[p] = exp2_poly2(x);
        } else {
            float x0, x1;
            unpack2(x, x0, x1);
            e[p] = pack2(ex2_approx(x0), ex2_approx(x1));
        }
        sum2 = add2(sum2, e[p]);
    }
    float s0, s1;
    unpack2(sum2, s0, s1);
    const float inv = __fdividef(keep, s0 + s1);
    const f32x2 inv2 = pack2(inv, inv);
    const int sw = row & 7;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float a, b;
            unpack2(mul2(e[4 * c + q], inv2), a, b);
            w[q] = pack_bf16(a, b);
        }
        *reinterpret_cast<uint4*>(row_base + ((c ^ sw) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

// The same for a PAIR of heads of dimension 64: u[0..31] are the token's logits under the first head's W, u[32..63]
// under the second head's.  Each group of 32 gets its own softmax.  Head b's feature vector, [softmax(+u_b),
// softmax(-u_b)], occupies block b of the tile (64 features): this thread's 32 values go to chunks 4 * kNeg .. 4 * kNeg + 3
// of the token's row in block b.  `tile_row` = start of the token's row in block 0; block 1 is kHalfTileBytes further.
template <bool kNeg>
__device__ __forceinline__ void softmax_pair_to_smem(float (&u)[kM], float keep0, float keep1, uint8_t* tile_row, int row)
{
    const int sw = row & 7;
#pragma unroll
    for (int b = 0; b < 2; ++b) {
        const int o = 32 * b;
        float m = kNeg ? min3(u[o], u[o + 1], u[o + 2]) : max3(u[o], u[o + 1], u[o + 2]);
#pragma unroll
        for (int j = 3; j < 31; j += 2) m = kNeg ? min3(m, u[o + j], u[o + j + 1]) : max3(m, u[o + j], u[o + j + 1]);
        m = kNeg ? fminf(m, u[o + 31]) : fmaxf(m, u[o + 31]);
        const float sL = kNeg ? -kLog2e : kLog2e;
        const float off = kNeg ? m * kLog2e : -m * kLog2e;
        const f32x2 scale = pack2(sL, sL), offset = pack2(off, off);
        f32x2 e[16];
        f32x2 sum2 = pack2(0.f, 0.f);
#pragma unroll
        for (int p = 0; p < 16; ++p) {
            const f32x2 x = fma2(pack2(u[o + 2 * p], u[o + 2 * p + 1]), scale, offset);
            if ((p & 3) == 3) {
                e[p] = exp2_poly2(x);
            } else {
                float x0, x1;
                unpack2(x, x0, x1);
                e[p] = pack2(ex2_approx(x0), ex2_approx(x1));
            }
            sum2 = add2(sum2, e[p]);
        }
        float s0, s1;
        unpack2(sum2, s0, s1);
        const float inv = __fdividef(b == 0 ? keep0 : keep1, s0 + s1);
        const f32x2 inv2 = pack2(inv, inv);
        uint8_t* dst = tile_row + b * kHalfTileBytes;
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
            uint32_t w[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                float x, y;
                unpack2(mul2(e[4 * cc + q], inv2), x, y);
                w[q] = pack_bf16(x, y);
            }
            const int chunk = (kNeg ? 4 : 0) + cc;
            *reinterpret_cast<uint4*>(dst + ((chunk ^ sw) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
}

// Read this thread's 64 logits (its TMEM lane, columns [col, col+64)).
__device__ __forceinline__ void load_logits(uint32_t taddr, float (&u)[kM])
{
    uint32_t r[kM];
    tmem_ld_x32(taddr, r);
    tmem_ld_x32(taddr + 32, r + 32);
    tmem_wait_ld();
#pragma unroll
    for (int j = 0; j < kM; ++j) u[j] = __uint_as_float(r[j]);
}

// Optional per-tile timestamps for tuning (compiled out unless LINATTN_TRACE is defined):
// trace[((cta * 4 + role) * kTraceTiles + tile) * 4 + event] = clock64.
#ifdef LINATTN_TRACE
constexpr int kTraceTiles = 64;
#define LA_TRACE(role, tile, ev)                                                                         \
    do {                                                                                                 \
        if (a.trace && (tile) < kTraceTiles && (threadIdx.x & 31) == 0)                                  \
            a.trace[(((size_t)blockIdx.x * 4 + (role)) * kTraceTiles + (tile)) * 4 + (ev)] = clock64(); \
    } while (0)
#define LA_TRACE_NS(role, tile, ev)                                                                             \
    do {                                                                                                        \
        if (a.trace && threadIdx.x == 0)                                                                        \
            a.trace[(((size_t)blockIdx.x * 4 + (role)) * kTraceTiles + (tile)) * 4 + (ev)] = (long long)globaltimer_ns(); \
    } while (0)
#define LA_TRACE_NS1(role, tile, ev)                                                                            \
    do {                                                                                                        \
        if (a.trace)                                                                                            \
            a.trace[(((size_t)blockIdx.x * 4 + (role)) * kTraceTiles + (tile)) * 4 + (ev)] = (long long)globaltimer_ns(); \
    } while (0)
#else
#define LA_TRACE(role, tile, ev) do { } while (0)
#define LA_TRACE_NS(role, tile, ev) do { } while (0)
#define LA_TRACE_NS1(role, tile, ev) do { } while (0)
#endif

// Shared-memory descriptor with the address field replaced: descriptors of one operand family differ
// only in their start address, so the constant part is built once.
__device__ __forceinline__ uint64_t desc_at(uint64_t base_desc, uint32_t smem_addr)
{
    return base_desc | (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
}

// U = X W (Eq. 6 logits) for one tile: A = X tile (K-major), B = W^T (K-major), D = 128 x 64 fp32.
// add = true: a second pass that adds X W_lo to the X W_hi already there (feature-map weights given in fp32 are held as
// a bf16 hi + lo pair, W = W_hi + W_lo to 2^-17 relative, so that fp32 weights run on the tensor cores too).
__device__ __forceinline__ void issue_logits_mma(uint32_t d_tmem, uint32_t x_smem, uint32_t w_smem, bool add = false)
{
    constexpr uint32_t idesc = make_idesc_bf16(kTile, kM, 0, 0);
    const uint64_t kmajor = make_desc_sw128(0, 16, 1024);
#pragma unroll
    for (int k = 0; k < kD / 16; ++k) {
        const uint64_t da = desc_at(kmajor, x_smem + (k >> 2) * kHalfTileBytes + (k & 3) * 32);
        const uint64_t db = desc_at(kmajor, w_smem + (k >> 2) * (kWBytes / 2) + (k & 3) * 32);
        mma_bf16_ss(d_tmem, da, db, idesc, (add || k > 0) ? 1u : 0u);
    }
}

// ======================================================================================================
// Shared-memory layout, barriers and per-CTA state common to all three kernels
// ======================================================================================================

// Key side: K and V have rings of their own.  A K slot is held from the issue of its load until the accumulation
// MMA has consumed the phi written over it (load latency + logits MMA + feature map + MMA).  V is needed only by that
// last MMA; its ring works in HALF tiles (64 tokens, the tokens of four of the MMA's eight K steps), each half with its
// own barriers, so that a half goes back to the producer as soon as its four K steps are done.  The rate of the key
// side is set by the slower of the two rings' loops, (hold time) / (slots): with whole-tile V slots, two of them gave
// (V load latency 2-3 us + MMA 0.8 us) / 2 = 1.75 us per tile against the 1.36 us per tile at which HBM delivers, and a
// third did not fit; five half tiles do (the feature-map weights are single-buffered to make the room).
constexpr int kKSlots = 4;
constexpr int kVHalves = 5;   // V ring: half tiles of 64 tokens x 128 columns (16 KB)
constexpr int kVLag = 1;      // the loads of V tile i are issued after that of K tile i + kVLag
constexpr int kQStages = 5;   // query side: stages of one Q tile (reused for phi(q) and then the output tile)
constexpr int kThreads = 512; // 16 warps
constexpr int kQPrefetchL2 = 3;   // fused kernel: Q tiles pulled into L2 while the CTA waits for S (measured: 2-3 best, 6+ slows the combine)

struct Smem {
    // key side
    static constexpr uint32_t kKV = kKSlots * kTileBytes;                 // K slots (each later holds phi), then the V half-tile slots
    static constexpr uint32_t kKW = kKV + kVHalves * kHalfTileBytes;      // W_k^T
    static constexpr uint32_t kOnes = kKW + kWBytes;                      // 1 KB of bf16 ones
    static constexpr uint32_t kKEnd = kOnes + 1024;
    // query side (overlays the key-side region)
    // [S | z] operand of the query side: per 64-feature block 144 rows of 128 bytes, rows 0-127 = S image [c][f],
    // rows 128-143 = z operand (hi, lo, zeros): ONE MMA of N = 144 per K step gives numerator and denominator
    static constexpr uint32_t kSZBlock = kHalfTileBytes + kZBlkBytes / 2; // 18 KB
    static constexpr uint32_t kQS = kQStages * kTileBytes;                // 2 blocks (36 KB)
    static constexpr uint32_t kQW = kQS + 2 * kSZBlock;                   // W_q^T (16 KB)
    static constexpr uint32_t kQEnd = kQW + kWBytes;
    static constexpr uint32_t kBars = kKEnd > kQEnd ? kKEnd : kQEnd;      // mbarriers, TMEM slot, abort word
    static constexpr uint32_t kTotal = kBars + 640 + 1024;                // + alignment slack
};

// mbarrier indices
enum : int {
    // key side
    K_FULL = 0, K_EMPTY = 4, K_PHIFULL = 8, K_VFULL = 12, K_VEMPTY = 18, K_UFULL = 24, K_UEMPTY = 26, K_WFULL = 28, K_WFREE = 29,
    K_ACCFULL = 30, K_ACCFREE = 32,
    // query side
    Q_FULL = 34, Q_EMPTY = 39, Q_PHIFULL = 44, Q_OFULL = 49, Q_UFULL = 54, Q_UEMPTY = 56, Q_DFULL = 58, Q_DEMPTY = 60,
    Q_SEGFULL = 62, Q_SEGFREE = 63, Q_WFULL = 65, Q_AFULL = 66,
    NBARS = 71
};
static_assert(kKSlots <= K_EMPTY - K_FULL && kVHalves <= K_VEMPTY - K_VFULL, "one mbarrier per ring slot: widen the enum before growing a ring");

struct Cta {
    uint8_t* smem;
    uint32_t sbase, bar0, tmem;
    int warp, lane;
    WaitCtx wc;
    __device__ __forceinline__ uint32_t bar(int i) const { return bar0 + 8u * (uint32_t)i; }
};

struct Args {
    float* partial;              // [slots][kE] partial (S, z) records, slot = cta + g; S as [c][f] (c = column of V, f = feature)
    float* state;                // [G][kE] combined S, z (fp32), same layout
    __nv_bfloat16* s_img;        // [G][128][128] bf16 image of S, [c][f]
    __nv_bfloat16* s_img_lo;     // or nullptr: bf16 image of what s_img leaves of S (S = hi + lo; the backward's operand pair)
    __nv_bfloat16* z_img;        // [G][kZBlkBytes / 2] bf16 operand image of z (hi, lo)
    uint32_t* err;               // error word
    uint32_t* sync;              // fused kernel: [0] CTAs that have left their last wait; [1 + 2g], [2 + 2g] arrivals at the two
                                 // per-head meeting points of (b,h) pair g.  All zero between launches (the kernel re-zeroes them)
    uint32_t wait_limit_us;      // bound of every device-side wait
    uint32_t arrive_extra;       // 0; a test sets 1, which makes every meeting point wait for one arrival more than will ever come
    const __nv_bfloat16* mix_src;  // Eq. 8: output of the softmax-attention branch [G][n][128], or nullptr (plain Eq. 5)
    float mix_r;                 // Eq. 8: the score r, already clipped into [0, 1]
    long long str_token, str_head, str_batch;  // element strides of q, k, v, out (and mix_src) between tokens, heads, batches
    int n, H, G;                 // tokens; heads per batch entry (H); units of work: (b,h) pairs, or pairs of heads when d = 64
    int heads_total;             // B * H
    int tiles_per_head;
    long long total_tiles;
#ifdef LINATTN_TRACE
    long long* trace;
#endif
};

// Common prologue: barrier init, TMEM allocation (512 columns, warp 9), abort word.
__device__ __forceinline__ Cta cta_setup(uint8_t* smem_raw, const Args& a, bool init_k, bool init_q)
{
    Cta c;
    c.smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    c.sbase = smem_u32(c.smem);
    uint64_t* bars = reinterpret_cast<uint64_t*>(c.smem + Smem::kBars);
    c.bar0 = smem_u32(bars);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(&bars[NBARS]);
    uint32_t* abort_word = tmem_slot + 1;
    c.warp = threadIdx.x >> 5;
    c.lane = threadIdx.x & 31;
    c.wc.err = a.err;
    c.wc.abort_smem = smem_u32(abort_word);
    c.wc.limit_us = a.wait_limit_us;
    if (threadIdx.x == 0) {
        *abort_word = 0u;
        if (init_k) {
            for (int i = 0; i < kKSlots; ++i) { mbar_init(c.bar(K_FULL + i), 1); mbar_init(c.bar(K_EMPTY + i), 1); mbar_init(c.bar(K_PHIFULL + i), 8); }
            for (int i = 0; i < kVHalves; ++i) { mbar_init(c.bar(K_VFULL + i), 1); mbar_init(c.bar(K_VEMPTY + i), 1); }
            for (int i = 0; i < 2; ++i) { mbar_init(c.bar(K_UFULL + i), 1); mbar_init(c.bar(K_UEMPTY + i), 8); }
            mbar_init(c.bar(K_WFULL), 1);
            mbar_init(c.bar(K_WFREE), 1);
            for (int i = 0; i < 2; ++i) { mbar_init(c.bar(K_ACCFULL + i), 1); mbar_init(c.bar(K_ACCFREE + i), 4); }
        }
        if (init_q) {
            for (int i = 0; i < kQStages; ++i) { mbar_init(c.bar(Q_FULL + i), 1); mbar_init(c.bar(Q_EMPTY + i), 1); mbar_init(c.bar(Q_PHIFULL + i), 8); mbar_init(c.bar(Q_OFULL + i), 4); mbar_init(c.bar(Q_AFULL + i), 1); }
            for (int i = 0; i < 2; ++i) { mbar_init(c.bar(Q_UFULL + i), 1); mbar_init(c.bar(Q_UEMPTY + i), 8); mbar_init(c.bar(Q_DFULL + i), 1); mbar_init(c.bar(Q_DEMPTY + i), 4); }
            mbar_init(c.bar(Q_SEGFULL), 1);
            mbar_init(c.bar(Q_SEGFREE), 1);
            mbar_init(c.bar(Q_WFULL), 1);
        }
        fence_mbar_init();
    }
    if (c.warp == 9) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    if (init_k)
        for (int i = threadIdx.x; i < 512; i += blockDim.x) reinterpret_cast<__nv_bfloat16*>(c.smem + Smem::kOnes)[i] = __float2bfloat16(1.0f);
    fence_proxy_async_smem();
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    c.tmem = *tmem_slot;
    return c;
}

__device__ __forceinline__ void cta_teardown(const Cta& c)
{
    tcgen05_fence_before();
    __syncthreads();
    if (c.warp == 9) tmem_dealloc(c.tmem, 512);
}

// Activations q, k, v, out as TMA sees them.  kLayout 0: [B][H][n][d], a rank-3 map (feature, token, b*H + h);
// kLayout 1: [B][n][H][d], a rank-4 map (feature, token, head, batch).  The rank-3 form is measurably faster
// (1.5 us per forward at B=1, H=12, n=32760), so the default layout keeps it.
template <int kLayout>
__device__ __forceinline__ void act_load(uint32_t dst, const void* tm, uint32_t bar, int x, int t, int g, int H)
{
    if (kLayout == 0) tma_load_3d(dst, tm, bar, x, t, g);
    else tma_load_4d(dst, tm, bar, x, t, g % H, g / H);
}
template <int kLayout>
__device__ __forceinline__ void act_store(const void* tm, uint32_t src, int x, int t, int g, int H)
{
    if (kLayout == 0) tma_store_3d(tm, src, x, t, g);
    else tma_store_4d(tm, src, x, t, g % H, g / H);
}
// The output tiles are stored with the L2 policy "evict last": the lines of the output then outlive, in L2, the lines of
// q that stream through next to them (measured: 2 us of 82 at B=1, H=12, n=32760), and whatever consumes the output next
// finds more of it on chip.
template <int kLayout>
__device__ __forceinline__ void act_store(const void* tm, uint32_t src, int x, int t, int g, int H, uint64_t policy)
{
    if (kLayout == 0) tma_store_3d_hint(tm, src, x, t, g, policy);
    else tma_store_4d_hint(tm, src, x, t, g % H, g / H, policy);
}
template <int kLayout>
__device__ __forceinline__ void act_prefetch_l2(const void* tm, int x, int t, int g, int H)
{
    if (kLayout == 0) tma_prefetch_l2_3d(tm, x, t, g);
    else tma_prefetch_l2_4d(tm, x, t, g % H, g / H);
}

// Where the two 64-feature blocks of a 128-token tile come from.
//   kPair = 0 (head dimension 128): features [0, 64) and [64, 128) of (b,h) pair g.
//   kPair = 1 (head dimension 64): the 64 features of heads 2g and 2g + 1, taken over the flattened (batch, head)
//   index: a PAIR of heads is processed as one 128-feature problem whose weight matrix, state S and normaliser z are
//   block-diagonal (the combine step zeroes the off-diagonal blocks of S, the z operand has one hi+lo column pair per
//   head), so every tensor-core shape, the shared-memory layout and the pipelines are those of d = 128.  If the number
//   of heads in all is odd, the last pair's second head does not exist: its loads start past the end of the tensor
//   (TMA fills zeros), its phi is forced to zero on the key side and its output block is not stored.
template <int kLayout, int kPair> struct Blocks {
    static __device__ __forceinline__ int head(int g, int blk) { return kPair ? 2 * g + blk : g; }
    static __device__ __forceinline__ int x(int blk) { return kPair ? 0 : 64 * blk; }
    static __device__ __forceinline__ void load(uint32_t dst, const void* tm, uint32_t bar, int blk, int t, int g, int H)
    {
        act_load<kLayout>(dst, tm, bar, x(blk), t, head(g, blk), H);
    }
    static __device__ __forceinline__ void store(const void* tm, uint32_t src, int blk, int t, int g, int H, uint64_t policy)
    {
        act_store<kLayout>(tm, src, x(blk), t, head(g, blk), H, policy);
    }
    static __device__ __forceinline__ void prefetch_l2(const void* tm, int blk, int t, int g, int H)
    {
        act_prefetch_l2<kLayout>(tm, x(blk), t, head(g, blk), H);
    }
    // which weight matrix (plane of the W^T tensor map) goes with (b,h) pair / pair of heads g
    static __device__ __forceinline__ int weights(int g, int H) { return (kPair ? 2 * g : g) % H; }
};

// ReLU kernel function, phi(x) = max(x, 0) element by element: applied in place to a 128 x 128 bf16 tile exactly as
// TMA left it in shared memory (element-wise, so the swizzled operand layout is kept); 256 threads, 128 bytes each.
// Rows past the end of the sequence were zero-filled by TMA and stay zero.
__device__ __forceinline__ void relu_tile_in_place(uint8_t* tile, int t)
{
#pragma unroll
    for (int j = 0; j < kTileBytes / (256 * 16); ++j) {
        uint4* p = reinterpret_cast<uint4*>(tile) + j * 256 + t;
        uint4 v = *p;
        asm("max.bf16x2 %0, %0, %1;" : "+r"(v.x) : "r"(0u));
        asm("max.bf16x2 %0, %0, %1;" : "+r"(v.y) : "r"(0u));
        asm("max.bf16x2 %0, %0, %1;" : "+r"(v.z) : "r"(0u));
        asm("max.bf16x2 %0, %0, %1;" : "+r"(v.w) : "r"(0u));
        *p = v;
    }
}

// ---- Meeting points of the fused kernel ---------------------------------------------------------------
// The one dependency of the forward: the query side of (b,h) pair g needs the S, z of ALL of g's keys.  The CTAs whose
// runs touch g meet twice, on two counters of their own: once when each has written its partial record of g (then
// each sums its share of the record), once when each has written its share of the sum (then each may load S, z).
// A CTA waits only for the few CTAs that share a head with it, not for the slowest of the whole grid.  The counters
// are zero when a launch starts and the kernel leaves them zero (the last CTA out clears them), so nothing about a
// launch is computed on the host and a launch recorded in a CUDA graph can be replayed.  Co-residency of the CTAs is
// what the cooperative launch guarantees.  Every wait is bounded and stops when the CTA's abort word is raised.

// First CTA whose run touches (b,h) pair g, and how many do.
__device__ __forceinline__ void head_ctas(const Args& a, long long P, int g, int& c0, int& cnt)
{
    c0 = (int)tile_owner((long long)g * a.tiles_per_head, a.total_tiles, P);
    cnt = (int)tile_owner((long long)(g + 1) * a.tiles_per_head - 1, a.total_tiles, P) - c0 + 1;
}
constexpr uint32_t kDrainWarps = 4;   // arrivals per CTA at a head's first meeting point (one per drain warp)
// Called by ONE thread after a warp- or CTA-level barrier: the release, together with that barrier, publishes what every
// thread that took part in it wrote before.
__device__ __forceinline__ void meet_arrive(uint32_t* ctr)
{
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(ctr) : "memory");
}
// Called by ONE thread, followed by a CTA-level barrier (or a shuffle) that hands the verdict to the others.
__device__ __forceinline__ bool meet_wait(const uint32_t* ctr, uint32_t target, const WaitCtx& wc)
{
    if (ld_acquire_gpu(ctr) >= target) return true;
    const uint64_t t0 = globaltimer_ns();
    uint32_t spins = 0;
    while (ld_acquire_gpu(ctr) < target) {
        if ((++spins & 15u) == 0u) {
            uint32_t ab;
            asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(ab) : "r"(wc.abort_smem) : "memory");
            if (ab != 0u || globaltimer_ns() - t0 > wc.limit_ns()) return false;
        }
    }
    return true;
}
__device__ __forceinline__ void raise_abort(const WaitCtx& wc, uint32_t code)
{
    atomicOr(wc.err, code);
    asm volatile("st.volatile.shared.u32 [%0], %1;" ::"r"(wc.abort_smem), "r"(1u) : "memory");
}

// ======================================================================================================
// Key side: partial S = sum phi(k)^T v and z = sum phi(k) over this CTA's tiles (Eq. 5 brackets, Eq. 6)
// ======================================================================================================

// kPhi: 0 = the Hedgehog feature map of Eq. 6; 1 = the ReLU kernel function (no projection, no softmax: the logits
// warp idles and warps 0-7 rectify the K tile in place).
// kSplit: 1 = the feature-map weights are a bf16 hi + lo pair (they were given in fp32): two logits passes per tile.  The
// low parts live in the last slot of the V ring (key side) and of the Q ring (query side), which then run with one
// slot fewer; a compile-time variant, so that the rings of the common case keep their compile-time sizes.
// arrive: fused kernel; every partial record written is announced at its head's first meeting point.
template <int kLayout, int kPhi, int kPair, int kSplit>
__device__ __forceinline__ void kside_phase(const Cta& c, const Args& a, const CUtensorMap* tmK, const CUtensorMap* tmV,
                                            const CUtensorMap* tmW, const CUtensorMap* tmWlo, bool arrive)
{
    constexpr int vh = kSplit ? kVHalves - 1 : kVHalves;   // half-tile slots of the V ring in use
    const uint32_t wlo_smem = c.sbase + Smem::kKV + (kVHalves - 1) * kHalfTileBytes;
    const uint32_t tmem_u = c.tmem;            // 2 x 64 columns of logits
    // two accumulator sets, alternating by segment, so that one drains while the next accumulates
    auto tmem_s = [&](int b) { return c.tmem + 128 + b * 144; };   // 128 columns: S[f][c], lane = f
    auto tmem_z = [&](int b) { return c.tmem + 256 + b * 144; };   // 16 columns: z[f] (all 16 equal)
    const int warp = c.warp, lane = c.lane;
    const uint32_t sbase = c.sbase;
    TileWalk w;
    w.init(a.total_tiles, a.tiles_per_head);

    if (warp == 8) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            tma_prefetch_desc(tmK);
            tma_prefetch_desc(tmV);
            tma_prefetch_desc(tmW);
        }
        Ring<kKSlots> r;
        Ring<vh> vr;
        TileWalk wv = w;                 // walks the V tiles, kVLag tiles behind the K tiles
        int issued = 0, issued_v = 0;    // K tiles and V half tiles whose loads have been issued so far
        bool ok = true;
        // one half tile of V: tokens [64 h, 64 h + 64) of tile wv, as two boxes of 64 columns (the map's box is 64 rows high);
        // a half that lies past the end of the sequence is zero-filled like any out-of-range row
        auto issue_v = [&]() {
            if (issued_v >= vh && !warp_wait(c.bar(K_VEMPTY + vr.s), vr.ph ^ 1u, c.wc, kErrProducer)) { ok = false; return; }
            if (lane == 0) {
                mbar_arrive_expect_tx(c.bar(K_VFULL + vr.s), kHalfTileBytes);
                const uint32_t vdst = sbase + Smem::kKV + vr.s * kHalfTileBytes;
                const int row = wv.lt * kTile + (issued_v & 1) * (kTile / 2);
                Blocks<kLayout, kPair>::load(vdst, tmV, c.bar(K_VFULL + vr.s), 0, row, wv.g, a.H);
                Blocks<kLayout, kPair>::load(vdst + kHalfTileBytes / 2, tmV, c.bar(K_VFULL + vr.s), 1, row, wv.g, a.H);
            }
            if (issued_v & 1) wv.next();
            ++issued_v;
            vr.next();
        };
        for (; !w.done() && ok; w.next(), r.next()) {
            if (w.i >= kKSlots && !warp_wait(c.bar(K_EMPTY + r.s), r.ph ^ 1u, c.wc, kErrProducer)) { ok = false; break; }
            LA_TRACE(0, w.i, 0);
            if (lane == 0) {
                mbar_arrive_expect_tx(c.bar(K_FULL + r.s), kTileBytes);
                const uint32_t kdst = sbase + r.s * kTileBytes;
                Blocks<kLayout, kPair>::load(kdst, tmK, c.bar(K_FULL + r.s), 0, w.lt * kTile, w.g, a.H);
                Blocks<kLayout, kPair>::load(kdst + kHalfTileBytes, tmK, c.bar(K_FULL + r.s), 1, w.lt * kTile, w.g, a.H);
            }
            issued = w.i + 1;
            if (w.i >= kVLag) {
                issue_v();
                if (ok) issue_v();
            }
        }
        while (ok && issued_v < 2 * issued) issue_v();
        if (!ok) {
            // unwinding after a time-out: let the copies already in flight land before the CTA moves on
            for (int i = (issued > kKSlots ? issued - kKSlots : 0); i < issued; ++i)
                mbar_wait(c.bar(K_FULL + i % kKSlots), (uint32_t)(i / kKSlots) & 1u, c.wc.limit_ns());
            for (int i = (issued_v > vh ? issued_v - vh : 0); i < issued_v; ++i)
                mbar_wait(c.bar(K_VFULL + i % vh), (uint32_t)(i / vh) & 1u, c.wc.limit_ns());
        }
    } else if (warp == 9) {
        // ---------------- logits MMA issuer: U = K W_k ----------------
        // This warp also fetches the head's W_k^T (one buffer): at a head boundary it waits for its own last logits MMAs
        // of the previous head, loads the next head's matrix (16 KB, an L2 hit after the first CTA) and goes on; the K
        // and V loads of the producer are not held up meanwhile.
        Ring<kKSlots> r;
        Ring<2> ur;
        for (; kPhi == 0 && !w.done(); w.next(), r.next(), ur.next()) {
            if (w.first()) {
                if (w.seg >= 1 && !warp_wait(c.bar(K_WFREE), (uint32_t)(w.seg - 1) & 1u, c.wc, kErrMmaLoad)) break;
                if (lane == 0) {
                    const int wi = Blocks<kLayout, kPair>::weights(w.g, a.H);
                    mbar_arrive_expect_tx(c.bar(K_WFULL), kSplit ? 2 * kWBytes : kWBytes);
                    tma_load_3d(sbase + Smem::kKW, tmW, c.bar(K_WFULL), 0, 0, wi);
                    tma_load_3d(sbase + Smem::kKW + kWBytes / 2, tmW, c.bar(K_WFULL), 64, 0, wi);
                    if (kSplit) {
                        tma_load_3d(wlo_smem, tmWlo, c.bar(K_WFULL), 0, 0, wi);
                        tma_load_3d(wlo_smem + kWBytes / 2, tmWlo, c.bar(K_WFULL), 64, 0, wi);
                    }
                }
                if (!warp_wait(c.bar(K_WFULL), (uint32_t)w.seg & 1u, c.wc, kErrMmaLoad)) break;
            }
            if (!warp_wait(c.bar(K_FULL + r.s), r.ph, c.wc, kErrMmaLoad)) break;
            LA_TRACE(1, w.i, 0);
            if (w.i >= 2 && !warp_wait(c.bar(K_UEMPTY + ur.s), ur.ph ^ 1u, c.wc, kErrMmaU)) break;
            tcgen05_fence_after();
            if (elect_one()) {
                issue_logits_mma(tmem_u + ur.s * kM, sbase + r.s * kTileBytes, sbase + Smem::kKW);
                if (kSplit) issue_logits_mma(tmem_u + ur.s * kM, sbase + r.s * kTileBytes, wlo_smem, true);
                mma_commit(c.bar(K_UFULL + ur.s));
                if (w.last()) mma_commit(c.bar(K_WFREE));
            }
            __syncwarp();
            LA_TRACE(1, w.i, 1);
        }
    } else if (warp == 10) {
        // ---------------- accumulation MMA issuer: S += phi^T V, z += phi^T 1 ----------------
        constexpr uint32_t idesc_s = make_idesc_bf16(kD, kD, 1, 1);   // A = phi^T (MN-major), B = V (MN-major)
        constexpr uint32_t idesc_z = make_idesc_bf16(kD, 16, 1, 0);   // B = ones (K-major, no swizzle)
        const uint64_t ones_desc = make_desc_noswizzle(sbase + Smem::kOnes, 128, 256);
        const uint64_t mnmajor = make_desc_sw128(0, kHalfTileBytes, 1024);        // phi^T: blocks of 64 features 16 KB apart
        const uint64_t mnmajor_v = make_desc_sw128(0, kHalfTileBytes / 2, 1024);  // V half tile: blocks of 64 columns 8 KB apart
        Ring<kKSlots> r;
        Ring<vh> vr;
        bool ok = true;
        for (; !w.done() && ok; w.next(), r.next()) {
            if (!warp_wait(c.bar(K_PHIFULL + r.s), r.ph, c.wc, kErrMmaPhi)) break;
            const bool first = w.first();
            const int b = w.seg & 1;
            if (first && w.seg >= 2 && !warp_wait(c.bar(K_ACCFREE + b), (uint32_t)((w.seg >> 1) - 1) & 1u, c.wc, kErrMmaAcc)) break;
            // the tile's eight K steps (16 tokens each) in two halves, each against its own half tile of V
            for (int h = 0; h < 2 && ok; ++h, vr.next()) {
                if (!warp_wait(c.bar(K_VFULL + vr.s), vr.ph, c.wc, kErrMmaLoad)) { ok = false; break; }
                if (h == 0) LA_TRACE(1, w.i, 2);
                tcgen05_fence_after();
                if (elect_one()) {
                    const uint32_t phi = sbase + r.s * kTileBytes, vt = sbase + Smem::kKV + vr.s * kHalfTileBytes;
#pragma unroll
                    for (int kk = 0; kk < kTile / 32; ++kk) {
                        const int k = h * (kTile / 32) + kk;
                        const uint64_t da = desc_at(mnmajor, phi + k * 2048);
                        const uint64_t db = desc_at(mnmajor_v, vt + kk * 2048);
                        const uint32_t acc = (first && k == 0) ? 0u : 1u;
                        mma_bf16_ss(tmem_s(b), da, db, idesc_s, acc);
                        mma_bf16_ss(tmem_z(b), da, ones_desc, idesc_z, acc);
                    }
                    mma_commit(c.bar(K_VEMPTY + vr.s));
                    if (h == 1) {
                        mma_commit(c.bar(K_EMPTY + r.s));
                        if (w.last()) mma_commit(c.bar(K_ACCFULL + b));
                    }
                }
                __syncwarp();
            }
            LA_TRACE(1, w.i, 3);
        }
    } else if (warp < 8 && kPhi == 1) {
        // ---------------- ReLU kernel function (warps 0-7) ----------------
        Ring<kKSlots> r;
        for (; !w.done(); w.next(), r.next()) {
            if (!warp_wait(c.bar(K_FULL + r.s), r.ph, c.wc, kErrSoftmaxU)) break;
            relu_tile_in_place(c.smem + r.s * kTileBytes, threadIdx.x);
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(c.bar(K_PHIFULL + r.s));
        }
    } else if (warp < 8) {
        // ---------------- feature map + drain (warps 0-7) ----------------
        const int half = warp >> 2;                       // 0: softmax(+U), 1: softmax(-U)
        const int row = (warp & 3) * 32 + lane;           // token within the tile == TMEM lane
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        Ring<kKSlots> r;
        Ring<2> ur;
        for (; !w.done(); w.next(), r.next(), ur.next()) {
            if (!warp_wait(c.bar(K_UFULL + ur.s), ur.ph, c.wc, kErrSoftmaxU)) break;
            if ((warp & 3) == 0) LA_TRACE(2 + half, w.i, 0);
            tcgen05_fence_after();
            float u[kM];
            load_logits(tmem_u + lane_base + ur.s * kM, u);
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(c.bar(K_UEMPTY + ur.s));
            if ((warp & 3) == 0) LA_TRACE(2 + half, w.i, 1);
            const float keep = (w.lt * kTile + row < a.n) ? 1.f : 0.f;
            if (kPair) {
                const float keep1 = (2 * w.g + 1 < a.heads_total) ? keep : 0.f;   // a last pair without a second head
                uint8_t* tile_row = c.smem + r.s * kTileBytes + row * 128;
                if (half == 0) softmax_pair_to_smem<false>(u, keep, keep1, tile_row, row);
                else softmax_pair_to_smem<true>(u, keep, keep1, tile_row, row);
            } else {
                uint8_t* dst = c.smem + r.s * kTileBytes + half * kHalfTileBytes + row * 128;
                if (half == 0) softmax_half_to_smem<false>(u, keep, dst, row);
                else softmax_half_to_smem<true>(u, keep, dst, row);
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(c.bar(K_PHIFULL + r.s));
            if ((warp & 3) == 0) LA_TRACE(2 + half, w.i, 2);
        }
    } else if (warp >= 12) {
        // ---------------- drain (warps 12-15): at the end of a segment the accumulators go to the partial record ---
        // thread = feature f = TMEM lane.  The record holds S as [c][f] (c = column of V), so that the 32 lanes
        // of a warp write 128 contiguous bytes per column; z follows.
        const int row = (warp & 3) * 32 + lane;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        for (; !w.done(); w.next()) {
            if (!w.last()) continue;
            const int b = w.seg & 1;
            if (!warp_wait(c.bar(K_ACCFULL + b), (uint32_t)(w.seg >> 1) & 1u, c.wc, kErrDrain)) break;
            tcgen05_fence_after();
            float* rec = a.partial + (size_t)(blockIdx.x + w.g) * kE;
            float* scol = rec + row;
#pragma unroll
            for (int c0 = 0; c0 < kD; c0 += 32) {
                uint32_t v[32];
                tmem_ld_x32(tmem_s(b) + lane_base + c0, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) scol[(size_t)(c0 + j) * kD] = __uint_as_float(v[j]);
            }
            uint32_t zr[2];
            tmem_ld_x2(tmem_z(b) + lane_base, zr);
            tmem_wait_ld();
            rec[kD * kD + row] = __uint_as_float(zr[0]);
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(c.bar(K_ACCFREE + b));
            // each of the four drain warps announces its quarter of the record by itself (kDrainWarps arrivals per CTA
            // and head): a CTA-level barrier here could be left waiting by a warp that gave up a wait
            if (arrive && lane == 0) meet_arrive(a.sync + 1 + 2 * w.g);
        }
    }
}

// ======================================================================================================
// Combine: S = sum of partials, z likewise, in CTA order; bf16 images for the query side
// ======================================================================================================

// Four consecutive elements (e4 .. e4+3, e4 a multiple of 4) of head g's record: sum the partials of the
// CTAs that touched the head in ascending CTA index (so the result does not depend on timing), store the
// fp32 state and the bf16 operand images.  All loads of a batch are issued before the first add.
// kPair (head dimension 64, two heads per record): the record's off-diagonal blocks (one head's features against the
// other head's columns) are dropped: zero in the bf16 image, so that the query side's product does not mix the heads;
// the fp32 state goes to the two heads' own records ([c][f] of 64 x 64, then z) and the z operand gets one hi+lo pair
// of rows per head (rows 0, 1: first head, features 0-63; rows 2, 3: second head, features 64-127; all else stays zero).
template <int kPair>
__device__ __forceinline__ void combine_quad(const Args& a, long long P, int g, int e4)
{
    const long long c0 = tile_owner((long long)g * a.tiles_per_head, a.total_tiles, P);
    const long long c1 = tile_owner((long long)(g + 1) * a.tiles_per_head - 1, a.total_tiles, P);
    const float4* p = reinterpret_cast<const float4*>(a.partial + (size_t)(c0 + g) * kE + e4);
    const int cnt = (int)(c1 - c0) + 1;
    constexpr int kBatch = 16;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int base = 0; base < cnt; base += kBatch) {
        float4 v[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u)
            v[u] = (base + u < cnt) ? __ldcg(p + (size_t)(base + u) * (kE / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            if (base + u < cnt) {
                acc.x += v[u].x;
                acc.y += v[u].y;
                acc.z += v[u].z;
                acc.w += v[u].w;
            }
        }
    }
    constexpr int kEh = 64 * 64 + 64;   // floats per head's state record when d = 64
    if (!kPair) *reinterpret_cast<float4*>(a.state + (size_t)g * kE + e4) = acc;
    const float r[4] = {acc.x, acc.y, acc.z, acc.w};
    if (e4 < kD * kD) {
        const int cc = e4 / kD, f0 = e4 % kD;   // column of V, first of the four features
        const bool keep = !kPair || (cc >> 6) == (f0 >> 6);
        uint2 packed;
        packed.x = keep ? pack_bf16(r[0], r[1]) : 0u;
        packed.y = keep ? pack_bf16(r[2], r[3]) : 0u;
        *reinterpret_cast<uint2*>(a.s_img + (size_t)g * kD * kD + e4) = packed;
        if (a.s_img_lo) {   // never with kPair (the backward's tensor-core kernels are d = 128 only)
            uint2 lo;
            lo.x = pack_bf16(r[0] - __uint_as_float(packed.x << 16), r[1] - __uint_as_float(packed.x & 0xffff0000u));
            lo.y = pack_bf16(r[2] - __uint_as_float(packed.y << 16), r[3] - __uint_as_float(packed.y & 0xffff0000u));
            *reinterpret_cast<uint2*>(a.s_img_lo + (size_t)g * kD * kD + e4) = lo;
        }
        if (kPair && keep && 2 * g + (cc >> 6) < a.heads_total)
            *reinterpret_cast<float4*>(a.state + (size_t)(2 * g + (cc >> 6)) * kEh + (cc & 63) * 64 + (f0 & 63)) = acc;
    } else {
        // z[f]: hi and lo bf16 parts into two rows of the K-major operand block of feature block f / 64
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const int f = e4 - kD * kD + t;
            const __nv_bfloat16 hi = __float2bfloat16_rn(r[t]);
            const __nv_bfloat16 lo = __float2bfloat16_rn(r[t] - __bfloat162float(hi));
            __nv_bfloat16* blk = a.z_img + (size_t)g * (kZBlkBytes / 2) + (f >> 6) * (16 * 64);
            const int fi = f & 63, chunk = fi >> 3, within = fi & 7;
            const int row = kPair ? 2 * (f >> 6) : 0;   // rows (row, row + 1); the swizzle term of a row below 8 is the row itself
            blk[row * 64 + ((chunk ^ row) << 3) + within] = hi;
            blk[(row + 1) * 64 + ((chunk ^ (row + 1)) << 3) + within] = lo;
            if (kPair && 2 * g + (f >> 6) < a.heads_total) a.state[(size_t)(2 * g + (f >> 6)) * kEh + 64 * 64 + fi] = r[t];
        }
    }
}

// ======================================================================================================
// Query side: o = phi(q) S / (phi(q) . z)  (Eq. 5, Eq. 6)
// ======================================================================================================

__device__ __forceinline__ void bulk_load_1d(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// wait_state: the S and z images are produced earlier in the same kernel (fused path); loads of them
// must wait at the head's second meeting point.  Otherwise they were written by a previous launch.
template <bool kMix, int kLayout, int kPhi, int kPair, int kSplit>
__device__ __forceinline__ void qside_phase(const Cta& c, const Args& a, const CUtensorMap* tmQ, const CUtensorMap* tmO,
                                            const CUtensorMap* tmW, const CUtensorMap* tmWlo, const CUtensorMap* tmS,
                                            const CUtensorMap* tmA, bool wait_state)
{
    constexpr int qs = kSplit ? kQStages - 1 : kQStages;   // slots of the Q ring in use
    const uint32_t wlo_smem = c.sbase + (kQStages - 1) * kTileBytes;
    const uint32_t tmem_u = c.tmem;  // 2 x 64 columns of logits
    auto tmem_num = [&](int db) { return c.tmem + 128 + db * 160; };   // 144 columns: num[token][c], c = 0..127, then
    auto tmem_den = [&](int db) { return c.tmem + 256 + db * 160; };   // 16 columns: [phi(q).z_hi, phi(q).z_lo, 0...]
    const int warp = c.warp, lane = c.lane;
    const uint32_t sbase = c.sbase;
    TileWalk w;
    w.init(a.total_tiles, a.tiles_per_head);

    if (warp == 8) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            tma_prefetch_desc(tmQ);
            tma_prefetch_desc(tmW);
            tma_prefetch_desc(tmS);
        }
        Ring<qs> r;
        int issued = 0;
        int state_g = -1;   // head whose S, z still have to be loaded (W already on its way)
        bool ok = true;
        auto load_state = [&]() {
            // S and z of head state_g; in the fused kernel they were written by other CTAs with ordinary
            // stores and become readable once every sharer of the head has arrived at its second meeting point
            if (wait_state) {
                int c0, cnt;
                head_ctas(a, gridDim.x, state_g, c0, cnt);
                int got = 1;
                if (lane == 0) {
                    got = meet_wait(a.sync + 2 + 2 * state_g, (uint32_t)cnt + a.arrive_extra, c.wc) ? 1 : 0;
                    if (!got) raise_abort(c.wc, kErrSeg);
                }
                if (!__shfl_sync(0xffffffffu, got, 0)) { ok = false; return; }
            }
            if (lane == 0) {
                if (wait_state) fence_proxy_async_all();
                mbar_arrive_expect_tx(c.bar(Q_SEGFULL), kTileBytes + kZBlkBytes);
                const __nv_bfloat16* zsrc = a.z_img + (size_t)state_g * (kZBlkBytes / 2);
                for (int blk = 0; blk < 2; ++blk) {
                    const uint32_t dst = sbase + Smem::kQS + blk * Smem::kSZBlock;
                    tma_load_3d(dst, tmS, c.bar(Q_SEGFULL), 64 * blk, 0, state_g);
                    bulk_load_1d(dst + kHalfTileBytes, zsrc + blk * (kZBlkBytes / 4), kZBlkBytes / 2, c.bar(Q_SEGFULL));
                }
            }
            state_g = -1;
        };
        for (; !w.done() && ok; w.next(), r.next()) {
            if (w.first()) {
                // A first piece of the run shorter than the ring ends before its S, z were asked for (that load is put
                // off until the ring is full): they are owed now, or the MMAs that free the single S buffer never run.
                if (state_g >= 0) load_state();
                if (!ok) break;
                if (w.seg >= 1 && !warp_wait(c.bar(Q_SEGFREE), (uint32_t)(w.seg - 1) & 1u, c.wc, kErrSeg)) break;
                if (kPhi == 0 && lane == 0) {
                    const int wi = Blocks<kLayout, kPair>::weights(w.g, a.H);
                    mbar_arrive_expect_tx(c.bar(Q_WFULL), kSplit ? 2 * kWBytes : kWBytes);
                    tma_load_3d(sbase + Smem::kQW, tmW, c.bar(Q_WFULL), 0, 0, wi);
                    tma_load_3d(sbase + Smem::kQW + kWBytes / 2, tmW, c.bar(Q_WFULL), 64, 0, wi);
                    if (kSplit) {
                        tma_load_3d(wlo_smem, tmWlo, c.bar(Q_WFULL), 0, 0, wi);
                        tma_load_3d(wlo_smem + kWBytes / 2, tmWlo, c.bar(Q_WFULL), 64, 0, wi);
                    }
                }
                state_g = w.g;
                // the first head's state may not exist yet: get the first Q tiles moving before waiting for it
                if (!(wait_state && w.seg == 0)) load_state();
            }
            if (state_g >= 0 && w.i >= qs) {
                if (wait_state && w.seg == 0) {
                    // The ring is full and S does not exist yet.  Once the CTAs of this head have drained their
                    // accumulators (first meeting point) HBM has little to do until the query side starts: use the time
                    // to pull the next Q tiles of this run into L2.
                    bool passed = false;
                    if (lane == 0) {
                        int c0, cnt;
                        head_ctas(a, gridDim.x, w.g, c0, cnt);
                        const uint64_t t0 = globaltimer_ns();
                        while (!(passed = ld_acquire_gpu(a.sync + 1 + 2 * w.g) >= kDrainWarps * (uint32_t)cnt)) {
                            __nanosleep(200);
                            uint32_t ab;
                            asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(ab) : "r"(c.wc.abort_smem) : "memory");
                            if (ab != 0u || globaltimer_ns() - t0 > c.wc.limit_ns()) break;
                        }
                        if (passed) {
                            TileWalk pw = w;
                            for (int j = 0; j < kQPrefetchL2 && !pw.done(); ++j, pw.next()) {
                                Blocks<kLayout, kPair>::prefetch_l2(tmQ, 0, pw.lt * kTile, pw.g, a.H);
                                Blocks<kLayout, kPair>::prefetch_l2(tmQ, 1, pw.lt * kTile, pw.g, a.H);
                            }
                        }
                    }
                    __syncwarp();
                }
                load_state();
            }
            if (!ok) break;
            if (w.i >= qs && !warp_wait(c.bar(Q_EMPTY + r.s), r.ph ^ 1u, c.wc, kErrProducer)) break;
            LA_TRACE(0, 24 + w.i, 0);
            if (lane == 0) {
                mbar_arrive_expect_tx(c.bar(Q_FULL + r.s), kTileBytes);
                Blocks<kLayout, kPair>::load(sbase + r.s * kTileBytes, tmQ, c.bar(Q_FULL + r.s), 0, w.lt * kTile, w.g, a.H);
                Blocks<kLayout, kPair>::load(sbase + r.s * kTileBytes + kHalfTileBytes, tmQ, c.bar(Q_FULL + r.s), 1, w.lt * kTile, w.g, a.H);
            }
            if (kMix) {
                // Eq. 8: the epilogue will read this tile's rows of the softmax branch's output straight from
                // global memory a few microseconds from now; start them on their way into L2 (the rows of a tile
                // are contiguous: 256 lines of 128 bytes, fewer in the ragged tail tile)
                const int rows = min(kTile, a.n - w.lt * kTile);
                for (int line = lane; line < rows * 2; line += 32) {   // two 128-byte lines per row of the tile (one per block)
                    const int blk = line & 1, hd = Blocks<kLayout, kPair>::head(w.g, blk);
                    if (kPair && hd >= a.heads_total) continue;
                    const __nv_bfloat16* p = a.mix_src + (size_t)(hd / a.H) * a.str_batch + (size_t)(hd % a.H) * a.str_head +
                                             ((size_t)w.lt * kTile + (line >> 1)) * a.str_token + Blocks<kLayout, kPair>::x(blk);
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
                }
            }
            issued = w.i + 1;
        }
        if (ok && state_g >= 0) load_state();
        if (wait_state && ok) {
            // This CTA has left the last of its waits on the meeting points.  The last CTA to say so clears the counters
            // for the next launch (nobody reads them any more: every CTA is past its last wait).
            uint32_t old = 0;
            if (lane == 0) old = atomicAdd(a.sync, 1u);
            if (__shfl_sync(0xffffffffu, old, 0) == gridDim.x - 1)
                for (int i = lane; i < 1 + 2 * a.G; i += 32) a.sync[i] = 0u;
        }
        if (!ok || issued < w.count) {
            // unwinding: let the copies already in flight land before the CTA moves on
            for (int i = (issued > qs ? issued - qs : 0); i < issued; ++i)
                mbar_wait(c.bar(Q_FULL + i % qs), (uint32_t)(i / qs) & 1u, c.wc.limit_ns());
        }
    } else if (warp == 9) {
        // ---------------- logits MMA issuer: U = Q W_q ----------------
        Ring<qs> r;
        Ring<2> ur;
        for (; kPhi == 0 && !w.done(); w.next(), r.next(), ur.next()) {
            if (w.first() && !warp_wait(c.bar(Q_WFULL), (uint32_t)w.seg & 1u, c.wc, kErrSeg)) break;
            if (!warp_wait(c.bar(Q_FULL + r.s), r.ph, c.wc, kErrMmaLoad)) break;
            LA_TRACE(1, 24 + w.i, 0);
            if (w.i >= 2 && !warp_wait(c.bar(Q_UEMPTY + ur.s), ur.ph ^ 1u, c.wc, kErrMmaU)) break;
            tcgen05_fence_after();
            if (elect_one()) {
                issue_logits_mma(tmem_u + ur.s * kM, sbase + r.s * kTileBytes, sbase + Smem::kQW);
                if (kSplit) issue_logits_mma(tmem_u + ur.s * kM, sbase + r.s * kTileBytes, wlo_smem, true);
                mma_commit(c.bar(Q_UFULL + ur.s));
            }
            __syncwarp();
            LA_TRACE(1, 24 + w.i, 1);
        }
    } else if (warp == 10) {
        // ---------------- numerator / denominator MMA issuer: num = phi(q) S, den = phi(q) . z ----------------
        constexpr uint32_t idesc_n = make_idesc_bf16(kTile, kD + 16, 0, 0);   // A = phi(q) (K-major), B = [S image [c][f]; z operand] (K-major)
        const uint64_t kmajor = make_desc_sw128(0, 16, 1024);
        const uint64_t mnmajor = make_desc_sw128(0, kHalfTileBytes, 1024);
        Ring<qs> r;
        Ring<2> dr;
        for (; !w.done(); w.next(), r.next(), dr.next()) {
            if (w.first() && !warp_wait(c.bar(Q_SEGFULL), (uint32_t)w.seg & 1u, c.wc, kErrSeg)) break;
            if (!warp_wait(c.bar(Q_PHIFULL + r.s), r.ph, c.wc, kErrMmaPhi)) break;
            if (w.i >= 2 && !warp_wait(c.bar(Q_DEMPTY + dr.s), dr.ph ^ 1u, c.wc, kErrMmaAcc)) break;
            LA_TRACE(1, 24 + w.i, 2);
            tcgen05_fence_after();
            if (elect_one()) {
                const uint32_t phi = sbase + r.s * kTileBytes;
#pragma unroll
                for (int k = 0; k < kD / 16; ++k) {
                    const uint64_t da = desc_at(kmajor, phi + (k >> 2) * kHalfTileBytes + (k & 3) * 32);
                    const uint64_t db = desc_at(kmajor, sbase + Smem::kQS + (k >> 2) * Smem::kSZBlock + (k & 3) * 32);
                    mma_bf16_ss(tmem_num(dr.s), da, db, idesc_n, k > 0);
                }
                mma_commit(c.bar(Q_DFULL + dr.s));
                if (w.last()) mma_commit(c.bar(Q_SEGFREE));   // this head's S, z and W may now be replaced
            }
            __syncwarp();
            LA_TRACE(1, 24 + w.i, 3);
        }
    } else if (warp == 11) {
        // ---------------- TMA stores of finished output tiles ----------------
        // The slot goes back to the producer as soon as the store has READ it (the write to global memory goes on
        // by itself): the query side runs at the rate at which slots come back, so every microsecond a slot is
        // held longer than needed costs throughput.
        if (lane == 0) tma_prefetch_desc(tmO);
        const uint64_t keep = policy_evict_last();
        Ring<qs> r;
        for (; !w.done(); w.next(), r.next()) {
            if (!warp_wait(c.bar(Q_OFULL + r.s), r.ph, c.wc, kErrStore)) break;
            if (lane == 0) {
                Blocks<kLayout, kPair>::store(tmO, sbase + r.s * kTileBytes, 0, w.lt * kTile, w.g, a.H, keep);
                if (!kPair || 2 * w.g + 1 < a.heads_total)   // an odd number of heads in all: the last pair has no second head
                    Blocks<kLayout, kPair>::store(tmO, sbase + r.s * kTileBytes + kHalfTileBytes, 1, w.lt * kTile, w.g, a.H, keep);
                bulk_commit_group();
                bulk_wait_group_read<0>();
                mbar_arrive(c.bar(Q_EMPTY + r.s));
            }
            __syncwarp();
            LA_TRACE(0, 24 + w.i, 1);
        }
        if (lane == 0) bulk_wait_group<0>();
    } else if (warp < 8 && kPhi == 1) {
        // ---------------- ReLU kernel function (warps 0-7): phi(q) in place in the tile's slot ----------------
        Ring<qs> r;
        for (; !w.done(); w.next(), r.next()) {
            if (!warp_wait(c.bar(Q_FULL + r.s), r.ph, c.wc, kErrSoftmaxU)) break;
            relu_tile_in_place(c.smem + r.s * kTileBytes, threadIdx.x);
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(c.bar(Q_PHIFULL + r.s));
        }
    } else if (warp < 8) {
        // ---------------- feature map (warps 0-7) ----------------
        const int half = warp >> 2;
        const int row = (warp & 3) * 32 + lane;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        Ring<qs> r;
        Ring<2> ur;
        for (; !w.done(); w.next(), r.next(), ur.next()) {
            if (!warp_wait(c.bar(Q_UFULL + ur.s), ur.ph, c.wc, kErrSoftmaxU)) break;
            if (warp == 0) LA_TRACE(2, 24 + w.i, 0);
            tcgen05_fence_after();
            float u[kM];
            load_logits(tmem_u + lane_base + ur.s * kM, u);
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(c.bar(Q_UEMPTY + ur.s));
            if (kPair) {
                uint8_t* tile_row = c.smem + r.s * kTileBytes + row * 128;
                if (half == 0) softmax_pair_to_smem<false>(u, 1.f, 1.f, tile_row, row);
                else softmax_pair_to_smem<true>(u, 1.f, 1.f, tile_row, row);
            } else {
                uint8_t* dst = c.smem + r.s * kTileBytes + half * kHalfTileBytes + row * 128;
                if (half == 0) softmax_half_to_smem<false>(u, 1.f, dst, row);
                else softmax_half_to_smem<true>(u, 1.f, dst, row);
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(c.bar(Q_PHIFULL + r.s));
            if (warp == 0) LA_TRACE(2, 24 + w.i, 1);
        }
    } else if (warp >= 12) {
        // ---------------- epilogue (warps 12-15): o = num / den, bf16, into the tile's slot ----------------
        const int row = (warp & 3) * 32 + lane;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const int sw = row & 7;
        constexpr bool mix = kMix;   // compile-time: the plain forward carries none of the blend's code
        // One finished tile: o = num / den (blended with the softmax branch's tile under Eq. 8), bf16, into slot `rs`.
        auto finish = [&](int rs, uint32_t rph, int ds) -> bool {
            // columns of the denominator operand: d = 128: [z_hi, z_lo]; paired heads: [z_hi, z_lo] of the first head, then of the second
            uint32_t dv[4];
            tmem_ld_x2(tmem_den(ds) + lane_base, dv);
            if (kPair) tmem_ld_x2(tmem_den(ds) + lane_base + 2, dv + 2);
            if (mix && !warp_wait(c.bar(Q_AFULL + rs), rph, c.wc, kErrEpilogue)) return false;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t v[64];
                tmem_ld_x32(tmem_num(ds) + lane_base + half * 64, v);
                tmem_ld_x32(tmem_num(ds) + lane_base + half * 64 + 32, v + 32);
                tmem_wait_ld();
                if (half == 1) {
                    // everything this tile needs from TMEM is in registers: release the accumulator
                    tcgen05_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(c.bar(Q_DEMPTY + ds));
                }
                const int dsel = kPair ? 2 * half : 0;   // paired heads: output block `half` belongs to head `half` of the pair
                const float inv = __fdividef(1.f, __uint_as_float(dv[dsel]) + __uint_as_float(dv[dsel + 1]));
                uint8_t* dst = c.smem + rs * kTileBytes + half * kHalfTileBytes + row * 128;
                if (!mix) {
                    const f32x2 inv2 = pack2(inv, inv);
#pragma unroll
                    for (int cc = 0; cc < 8; ++cc) {
                        uint32_t o[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            float x, y;
                            unpack2(mul2(pack2(__uint_as_float(v[8 * cc + 2 * q]), __uint_as_float(v[8 * cc + 2 * q + 1])), inv2), x, y);
                            o[q] = pack_bf16(x, y);
                        }
                        *reinterpret_cast<uint4*>(dst + ((cc ^ sw) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                    }
                } else {
                    // o = r * softmax branch + (1 - r) * num / den, in fp32, rounded once
                    const float lin = (1.f - a.mix_r) * inv;
                    const f32x2 lin2 = pack2(lin, lin), r2 = pack2(a.mix_r, a.mix_r);
#pragma unroll
                    for (int cc = 0; cc < 8; ++cc) {
                        const uint4 av = *reinterpret_cast<const uint4*>(dst + ((cc ^ sw) << 4));
                        const uint32_t aw4[4] = {av.x, av.y, av.z, av.w};
                        uint32_t o[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const f32x2 soft = pack2(__uint_as_float(aw4[q] << 16), __uint_as_float(aw4[q] & 0xffff0000u));
                            float x, y;
                            unpack2(fma2(pack2(__uint_as_float(v[8 * cc + 2 * q]), __uint_as_float(v[8 * cc + 2 * q + 1])), lin2,
                                         mul2(soft, r2)), x, y);
                            o[q] = pack_bf16(x, y);
                        }
                        *reinterpret_cast<uint4*>(dst + ((cc ^ sw) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                    }
                }
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(c.bar(Q_OFULL + rs));
            return true;
        };
        Ring<qs> r;
        Ring<2> dr;
        // Eq. 8 (mixed attention): once the tensor core is done with phi(q) in a slot (that is what Q_DFULL says), the
        // tile of the softmax branch's output is brought into the very same slot by TMA (its lines are already on their
        // way into L2), blended in place and stored from there.  The blend of a tile runs one tile late, so that the
        // copy's latency passes under the blend of the tile before it instead of in front of its own.
        int prev_rs = -1, prev_ds = 0;
        uint32_t prev_rph = 0;
        bool ok = true;
        for (; !w.done(); w.next(), r.next(), dr.next()) {
            if (!warp_wait(c.bar(Q_DFULL + dr.s), dr.ph, c.wc, kErrEpilogue)) { ok = false; break; }
            if (warp == 12) LA_TRACE(3, 24 + w.i, 0);
            tcgen05_fence_after();
            if (mix) {
                if (warp == 12 && lane == 0) {
                    mbar_arrive_expect_tx(c.bar(Q_AFULL + r.s), kTileBytes);
                    Blocks<kLayout, kPair>::load(sbase + r.s * kTileBytes, tmA, c.bar(Q_AFULL + r.s), 0, w.lt * kTile, w.g, a.H);
                    Blocks<kLayout, kPair>::load(sbase + r.s * kTileBytes + kHalfTileBytes, tmA, c.bar(Q_AFULL + r.s), 1, w.lt * kTile, w.g, a.H);
                }
                if (prev_rs >= 0 && !finish(prev_rs, prev_rph, prev_ds)) { ok = false; break; }
                prev_rs = r.s;
                prev_rph = r.ph;
                prev_ds = dr.s;
            } else if (!finish(r.s, r.ph, dr.s)) { ok = false; break; }
            if (warp == 12) LA_TRACE(3, 24 + w.i, 1);
        }
        if (mix && prev_rs >= 0) {
            // the last tile; after a wait that gave up, only so that the copy in flight has landed before the CTA moves on
            if (ok) finish(prev_rs, prev_rph, prev_ds);
            else if (warp == 12) mbar_wait(c.bar(Q_AFULL + prev_rs), prev_rph, c.wc.limit_ns());
        }
    }
}

// ======================================================================================================
// Kernels
// ======================================================================================================

template <int kLayout, int kPhi, int kPair, int kSplit>
__global__ void __launch_bounds__(kThreads, 1)
kside_tc(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
         const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmWlo, const Args a)
{
    extern __shared__ uint8_t smem_raw[];
    const Cta c = cta_setup(smem_raw, a, true, false);
    kside_phase<kLayout, kPhi, kPair, kSplit>(c, a, &tmK, &tmV, &tmW, &tmWlo, false);
    cta_teardown(c);
}

// grid = (ceil(kE / 4 / 256), G)
template <int kPair>
__global__ void __launch_bounds__(256) combine_tc(const Args a, long long P)
{
    const int q4 = blockIdx.x * 256 + threadIdx.x;
    if (q4 < kE / 4) combine_quad<kPair>(a, P, blockIdx.y, q4 * 4);
}

template <bool kMix, int kLayout, int kPhi, int kPair, int kSplit>
__global__ void __launch_bounds__(kThreads, 1)
qside_tc(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmO,
         const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmWlo,
         const __grid_constant__ CUtensorMap tmS, const __grid_constant__ CUtensorMap tmA, const Args a)
{
    extern __shared__ uint8_t smem_raw[];
    const Cta c = cta_setup(smem_raw, a, false, true);
    qside_phase<kMix, kLayout, kPhi, kPair, kSplit>(c, a, &tmQ, &tmO, &tmW, &tmWlo, &tmS, &tmA, false);
    cta_teardown(c);
}

// The whole forward in one cooperative launch of P <= #SMs persistent CTAs.
template <bool kMix, int kLayout, int kPhi, int kPair, int kSplit>
__global__ void __launch_bounds__(kThreads, 1)
linattn_fused_tc(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                 const __grid_constant__ CUtensorMap tmWk, const __grid_constant__ CUtensorMap tmWklo,
                 const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmO,
                 const __grid_constant__ CUtensorMap tmWq, const __grid_constant__ CUtensorMap tmWqlo,
                 const __grid_constant__ CUtensorMap tmS, const __grid_constant__ CUtensorMap tmA, const Args a)
{
    extern __shared__ uint8_t smem_raw[];
    LA_TRACE_NS(0, 60, 0);
    const Cta c = cta_setup(smem_raw, a, true, true);
    LA_TRACE_NS(0, 60, 1);
    kside_phase<kLayout, kPhi, kPair, kSplit>(c, a, &tmK, &tmV, &tmWk, &tmWklo, true);
    // every role is done with the key-side buffers; the partials of this CTA are written and announced
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    LA_TRACE_NS(0, 60, 2);
    constexpr int kHoleThreads = 14 * 32;
    if (c.warp != 8 && c.warp != 9) {
        // Every warp but the producer and the logits issuer (which go straight on: Q tiles, W_q and the first logits do not
        // depend on S): for every head this CTA's run touches, wait at the head's first meeting point, sum this CTA's
        // share of the head's record, announce it at the second.  With 448 threads a share of a twelfth of a record (344
        // groups of four) is one group per thread: ONE round of loads from L2 instead of two (the step took 4 us with the
        // six warps that are idle anyway; the feature-map warps have nothing urgent to do until S exists either).
        __shared__ uint32_t met;
        const long long P = gridDim.x;
        const int it = c.warp < 8 ? (int)threadIdx.x : (int)threadIdx.x - 64;
        TileWalk w;
        w.init(a.total_tiles, a.tiles_per_head);
        bool ok = true;
        while (!w.done() && ok) {
            const int g = w.g;
            int c0, cnt;
            head_ctas(a, P, g, c0, cnt);
            if (it == 0) {
                met = meet_wait(a.sync + 1 + 2 * g, kDrainWarps * (uint32_t)cnt + a.arrive_extra, c.wc) ? 1u : 0u;
                if (!met) raise_abort(c.wc, kErrGrid);
            }
            named_barrier_sync(1, kHoleThreads);
            ok = met != 0u;
            if (it == 0 && w.seg == 0) LA_TRACE_NS1(0, 60, 3);
            if (ok) {
                const int j = (int)blockIdx.x - c0;
                const int lo = j * (kE / 4) / cnt, hi = (j + 1) * (kE / 4) / cnt;   // this CTA's share: float4 groups [lo, hi)
                for (int x = lo + it; x < hi; x += kHoleThreads) combine_quad<kPair>(a, P, g, x * 4);
            }
            named_barrier_sync(1, kHoleThreads);   // the share is written (and `met` has been read by everybody)
            if (it == 0 && ok) meet_arrive(a.sync + 2 + 2 * g);
            if (it == 0 && w.seg == 0) LA_TRACE_NS1(0, 61, 0);
            do w.next(); while (!w.done() && w.g == g);
        }
        if (it == 0) LA_TRACE_NS1(0, 61, 1);
    }
    qside_phase<kMix, kLayout, kPhi, kPair, kSplit>(c, a, &tmQ, &tmO, &tmWq, &tmWqlo, &tmS, &tmA, true);
    LA_TRACE_NS(0, 61, 2);
    cta_teardown(c);
    LA_TRACE_NS(0, 61, 3);
}

// W [H][128 d][64 j] (any supported type) -> W^T bf16 [H][64 j][128 d]; per_head == 0 replicates one matrix.
// bf16 hi part of w, or (lo != 0) the bf16 rounding of what the hi part leaves: w = hi + lo to 2^-17 relative.
__device__ __forceinline__ __nv_bfloat16 bf16_part(float w, int lo)
{
    const __nv_bfloat16 hi = __float2bfloat16_rn(w);
    return lo ? __float2bfloat16_rn(w - __bfloat162float(hi)) : hi;
}
template <typename T>
static __global__ void transpose_weights_bf16(const T* __restrict__ src, __nv_bfloat16* __restrict__ dst, int H, int per_head, int lo)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)H * kM * kD) return;
    const int h = (int)(i / (kM * kD)), rem = (int)(i % (kM * kD)), j = rem / kD, dd = rem % kD;
    const size_t s = (size_t)(per_head ? h : 0) * kD * kM + (size_t)dd * kM + j;
    dst[i] = bf16_part((float)src[s], lo);
}

// Head dimension 64: the weight image of a PAIR of heads, as the logits MMA of the d = 128 kernels wants it.
// dst [H][64 j'][128 d'] bf16, plane h0 for the pair (h0, h1 = (h0 + 1) mod H):
//   rows  0..31: W_{h0}^T (32 x 64) in columns 0..63,   zeros in columns 64..127
//   rows 32..63: zeros in columns 0..63,                W_{h1}^T in columns 64..127
// so that [x_{h0}, x_{h1}] (128 features) times its transpose gives [u_{h0} (32 logits), u_{h1} (32 logits)].
// src: W [H][64 d][32 j] (any supported type); per_head == 0: one matrix for every head.
template <typename T>
static __global__ void pair_weights_bf16(const T* __restrict__ src, __nv_bfloat16* __restrict__ dst, int H, int per_head, int lo)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)H * kM * kD) return;
    const int h0 = (int)(i / (kM * kD)), rem = (int)(i % (kM * kD)), jp = rem / kD, dp = rem % kD;
    const int blk = jp >> 5;   // which head of the pair this row of logits belongs to
    float v = 0.f;
    if ((dp >> 6) == blk) {
        const int h = per_head ? (h0 + blk) % H : 0;
        v = (float)src[(size_t)h * 64 * 32 + (size_t)(dp & 63) * 32 + (jp & 31)];
    }
    dst[i] = bf16_part(v, lo);
}

}  // namespace tc
}  // namespace linattn
