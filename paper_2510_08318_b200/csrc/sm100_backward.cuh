// Tensor-core kernels (tcgen05 + TMEM + TMA) for the gradients of linear attention with the Hedgehog feature map
// (what Eq. 14 back-propagates through Eq. 5 and Eq. 6), bf16 storage, head dimension 128.
//
// With dO the incoming gradient, den_i = phi(q_i).z, o_i = phi(q_i) S / den_i:
//     dnum_i = dO_i / den_i                  dden_i = -(dO_i . o_i) / den_i
//     dphi(q_i) = S dnum_i + dden_i z        dS = sum_i phi(q_i)^T dnum_i       dz = sum_i dden_i phi(q_i)
//     dphi(k_j) = dS v_j + dz                dv_j = dS^T phi(k_j)
//     du = p+ (.) (dphi+ - p+ . dphi+) - p- (.) (dphi- - p- . dphi-)       dx = du W^T       dW += x^T du
//
// Two kernels of persistent CTAs, each walking its contiguous run of 128-token tiles.  Every matrix product is a
// tcgen05.mma with fp32 accumulators in TMEM.  Warp-specialised: eight element-wise warps (thread = (token, half of the
// features)), a warp that issues the products and the copies they wait for, a warp that stores the staged results and
// requests the tile that follows into a buffer once its store has read it; mbarriers both ways.  Within a head the tiles
// are software-pipelined two deep: the tile that feeds the logits is double-buffered, the next tile's logits and first
// products are issued around this tile's last tensor-core stage, and this tile's results leave tensor memory after the
// next tile's feature map (the schedule is written out above qside_bwd_tc):
//
//   qside_bwd_tc : U = Q W_q -> phi(q), den = phi . z -> T = dO S^T -> dO . o = (T . phi) / den ->
//                  dphi = (T - (dO . o) z) / den, dS += (phi / den)^T dO, dz += (phi / den)^T (dden den) -> du ->
//                  dq = du W_q^T (TMA store), dW_q += Q^T du
//   kside_bwd_tc : U = K W_k -> phi(k) -> dphi = V dS^T (+ dz) -> du -> dk = du W_k^T (TMA store), dW_k += K^T du,
//                  dv = phi dS (TMA store)
//
// Operands that carry a difference of nearly equal terms downstream are kept exact or split into bf16 hi + lo
// parts: S and dS are hi + lo images written by the combine kernels (two passes each); dnum = dO / den is never
// formed: its per-token factor 1 / den is applied to the accumulator (dphi) or folded into phi (dS), so that the
// dO tile, exact in bf16, is the operand.  phi, phi / den and du are single bf16 operands, as phi is in the forward.
// Accumulators that live across tiles (dS, dW) are written as one record per (CTA, head) and summed in CTA
// order by the combine kernels, so the gradients are bit-reproducible.  Every wait is bounded.
#pragma once
#include "sm100_kernels.cuh"

namespace linattn {
namespace tc {

// Warps 0-7 do the element-wise work (thread = (token, half of the features)); warp 8 issues the tensor-core products
// and the copies they wait for; warp 9 stores the staged results and, once a store has read its buffer, requests the
// tile that comes into it next (a wait the issuer must not sit in); warps 10-11 only complete the group of four, which
// gives most of its registers to the element-wise warps.
constexpr int kBwdThreads = 384;
constexpr int kBwdCompute = 256;
constexpr int kBwdIssuer = 8;
// Registers per thread after the split.  A CTA of 384 threads starts with 168 each, and what the three warp groups hold
// afterwards can only come out of that: 2 x element-wise + issuer <= 3 x 168 (a request beyond it would wait for ever).
constexpr int kBwdRegsCompute = 216, kBwdRegsIssuer = 72;
static_assert(2 * kBwdRegsCompute + kBwdRegsIssuer <= 3 * 168 && kBwdRegsCompute % 8 == 0 && kBwdRegsIssuer % 8 == 0, "register split");
constexpr int kWRec = kM * kD;   // floats per weight-gradient record, stored [j][c]

struct BwdArgs {
    float* part_state;     // [slots][kE]: per (CTA, head) sums of dS as [c][f], then dz   (query side writes)
    float* part_w;         // [slots][kWRec]: per (CTA, head) sums of dW as [j][c]
    const float* state;    // [G][kE]: query side: S as [c][f], then z; key side: dS as [c][f], then dz
    uint32_t* err;
    // Eq. 8 (mixed attention): the linear branch's incoming gradient is lin_scale * dout, lin_scale = 1 - r^ (1 for the
    // plain operator); with mix_a (the softmax branch's output, laid out like q) the query side also sums
    // dout . (a - o) into part_dr [CTA], the terms of dL/dr
    const __nv_bfloat16* mix_a;
    float* part_dr;
    float lin_scale;
    long long str_token, str_head, str_batch;   // element strides of the activations (for the reads of mix_a)
    int n, H, G, tiles_per_head;
    long long total_tiles;
    uint32_t wait_limit_us;   // bound of every wait in the kernel
    int test_unmet;           // tests of the time-out path only: warp 0 leaves out one arrival (the operands of its CTA's first tile)
#ifdef LINATTN_TRACE
    long long* trace;      // tuning builds: [CTA][tile < 8][16] clock64 stamps of the stages of a tile
#endif
};

#ifdef LINATTN_TRACE
#define LB_TRACE(ev)                                                                                                  \
    do {                                                                                                              \
        if (a.trace && threadIdx.x == 0 && w.i < 8) a.trace[((size_t)blockIdx.x * 8 + w.i) * 16 + (ev)] = clock64(); \
    } while (0)
#define LB_TRACE_K(ev)                                                                                                \
    do {                                                                                                              \
        if (a.trace && threadIdx.x == 0 && w.i < 8) a.trace[((size_t)(148 + blockIdx.x) * 8 + w.i) * 16 + (ev)] = clock64(); \
    } while (0)
#define LB_TRACE_I(region, ev)                                                                                        \
    do {                                                                                                              \
        if (a.trace && one && w.i < 8) a.trace[((size_t)((region) * 148 + blockIdx.x) * 8 + w.i) * 16 + (ev)] = clock64(); \
    } while (0)
#else
#define LB_TRACE(ev) do { } while (0)
#define LB_TRACE_K(ev) do { } while (0)
#define LB_TRACE_I(region, ev) do { } while (0)
#endif

// Shared memory, both kernels: two buffers for the tile that feeds the logits (the next tile's is fetched while this
// tile is worked on), one for the other input tile, the staging tile, the hi and lo images, the weights and the du
// tile: 224 KB, then the small block below.  The total is the 227 KB a CTA may have, to within 448 bytes: the
// kernels leave with an error if the base of the dynamic array is not aligned well enough for that.
struct BwdSmemQ {   // query side
    static constexpr uint32_t kX0 = 0;                       // Q tile, even tiles of the run
    static constexpr uint32_t kX1 = kX0 + kTileBytes;        // Q tile, odd tiles
    static constexpr uint32_t kG = kX1 + kTileBytes;         // dO tile
    static constexpr uint32_t kP = kG + kTileBytes;          // phi(q) / den -> dq staging
    static constexpr uint32_t kShi = kP + kTileBytes;        // S image [c][f], hi part
    static constexpr uint32_t kSlo = kShi + kTileBytes;      // lo part
    static constexpr uint32_t kW = kSlo + kTileBytes;        // W_q^T [64][128]
    static constexpr uint32_t kDu = kW + kWBytes;            // du tile [128][64] bf16 (16 KB)
    static constexpr uint32_t kRed = kDu;                    // at the end of a head (du consumed): 16 x 128 floats, dz sums of the token groups
    static constexpr uint32_t kMisc = kDu + kWBytes;
};
struct BwdSmemK {   // key side
    static constexpr uint32_t kX0 = 0;                       // K tile, even tiles of the run
    static constexpr uint32_t kX1 = kX0 + kTileBytes;        // K tile, odd tiles
    static constexpr uint32_t kV = kX1 + kTileBytes;         // V tile
    static constexpr uint32_t kP = kV + kTileBytes;          // phi(k) -> dv staging -> dk staging
    static constexpr uint32_t kShi = kP + kTileBytes;        // dS image [c][f], hi part
    static constexpr uint32_t kSlo = kShi + kTileBytes;
    static constexpr uint32_t kW = kSlo + kTileBytes;        // W_k^T [64][128]
    static constexpr uint32_t kDu = kW + kWBytes;            // du tile [128][64] bf16
    static constexpr uint32_t kMisc = kDu + kWBytes;
};
// misc block: z / dz vector, per-token scalars, barriers, TMEM slot, abort word
struct BwdMisc {
    static constexpr uint32_t kVec = 0;           // 128 floats: z (query side) or dz (key side)
    static constexpr uint32_t kA = 512;           // 2 x 128 floats: den halves
    static constexpr uint32_t kB = 1536;          // 2 x 128 floats: (dO . o) halves; then, in the first 128, dden den of the tile
    static constexpr uint32_t kBars = 2560;       // 12 mbarriers, TMEM slot, abort word
    static constexpr uint32_t kBytes = 2560 + 112;
};
constexpr uint32_t kBwdSmemQ = BwdSmemQ::kMisc + BwdMisc::kBytes;
constexpr uint32_t kBwdSmemK = BwdSmemK::kMisc + BwdMisc::kBytes;
static_assert(kBwdSmemQ <= 232448 && kBwdSmemK <= 232448, "a CTA has 227 KB of shared memory");

// mbarriers.  Copies: BW_X0 / BW_X1 the two buffers of the tile that feeds the logits, BW_IN2 the other input tile,
// BW_SEG the head's images and weights.  Issuer -> element-wise warps: BW_LFULL logits, BW_TFULL the product with the
// images, BW_G1 / BW_GFULL the first part / all of the tile's last tensor-core stage.  Element-wise warps -> issuer (one
// arrival per warp): BW_OPS1 / BW_OPS the first / all operands of the last stage are written, BW_STAGED1 / BW_STAGED
// results have been staged for their stores.
enum : int {
    BW_X0 = 0, BW_X1 = 1, BW_IN2 = 2, BW_SEG = 3, BW_LFULL = 4, BW_TFULL = 5, BW_G1 = 6, BW_GFULL = 7,
    BW_OPS1 = 8, BW_OPS = 9, BW_STAGED1 = 10, BW_STAGED = 11, BW_NBARS = 12
};

struct BwdCta {
    uint8_t* smem;
    uint32_t sbase, bar0, tmem;
    float* misc;
    WaitCtx wc;
    __device__ __forceinline__ uint32_t bar(int i) const { return bar0 + 8u * (uint32_t)i; }
};

// The layout above leaves no room for rounding the base of the dynamic shared memory up to the 1024 bytes the swizzled
// tiles need.  These kernels have no static shared memory, so their dynamic array starts at the CTA's window, which is
// so aligned; this check (the same verdict in every thread, before any barrier or allocation) makes a launch whose
// array came out otherwise report it and leave instead of writing past its end.
__device__ __forceinline__ bool bwd_smem_fits(const uint8_t* smem_raw, uint32_t need, uint32_t* err)
{
    uint32_t have;
    asm volatile("mov.u32 %0, %%dynamic_smem_size;" : "=r"(have));
    const uint32_t pad = (1024u - (smem_u32(smem_raw) & 1023u)) & 1023u;
    if (pad + need <= have) return true;
    if (threadIdx.x == 0) atomicOr(err, kErrSmem);
    return false;
}

__device__ __forceinline__ BwdCta bwd_setup(uint8_t* smem_raw, uint32_t misc_off, uint32_t* err, uint32_t wait_limit_us)
{
    BwdCta c;
    c.smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    c.sbase = smem_u32(c.smem);
    c.misc = reinterpret_cast<float*>(c.smem + misc_off);
    uint64_t* bars = reinterpret_cast<uint64_t*>(c.smem + misc_off + BwdMisc::kBars);
    c.bar0 = smem_u32(bars);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(&bars[BW_NBARS]);
    uint32_t* abort_word = tmem_slot + 1;
    c.wc.err = err;
    c.wc.abort_smem = smem_u32(abort_word);
    c.wc.limit_us = wait_limit_us;
    if (threadIdx.x == 0) {
        *abort_word = 0u;
        for (int i = 0; i < BW_NBARS; ++i) mbar_init(c.bar(i), i >= BW_OPS1 ? kBwdCompute / 32 : 1);
        fence_mbar_init();
    }
    if ((threadIdx.x >> 5) == 1) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    fence_proxy_async_smem();
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    c.tmem = *tmem_slot;
    return c;
}

__device__ __forceinline__ void bwd_teardown(const BwdCta& c)
{
    tcgen05_fence_before();
    __syncthreads();
    if ((threadIdx.x >> 5) == 1) tmem_dealloc(c.tmem, 512);
}

// Barrier of the element-wise warps.
__device__ __forceinline__ void cbar() { named_barrier_sync(1, kBwdCompute); }
// The same with a verdict: false for everybody if any thread brings false (a wait of its own that gave up).
__device__ __forceinline__ bool cbar_and(bool ok) { return named_barrier_and(1, kBwdCompute, ok); }

// All element-wise threads wait (bounded) for the barrier's phase and meet; the verdict is the same for every one of
// them, so the stage loop never leaves some of them behind at a barrier.  `ok` carries the verdict of earlier waits
// that did not meet (wait_only).
__device__ __forceinline__ bool compute_wait(const BwdCta& c, int b, uint32_t& phase, uint32_t code, bool ok = true)
{
    const bool mine = warp_wait(c.bar(b), phase, c.wc, code);
    phase ^= 1u;
    const bool all = cbar_and(ok && mine);
    tcgen05_fence_after();
    return all;
}
__device__ __forceinline__ bool wait_only(const BwdCta& c, int b, uint32_t& phase, uint32_t code)
{
    const bool mine = warp_wait(c.bar(b), phase, c.wc, code);
    phase ^= 1u;
    tcgen05_fence_after();
    return mine;
}
// What a warp has written (shared memory for the tensor core or a store, tensor memory reads done) is announced to the issuer.
__device__ __forceinline__ void warp_announce(const BwdCta& c, int b)
{
    fence_proxy_async_smem();
    tcgen05_fence_before();
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(c.bar(b));
}

// Byte offset of 16-byte chunk `ch` (8 bf16) of row `row` inside a 64-column block of a TMA tile (128-byte swizzle).
__device__ __forceinline__ uint32_t sw_chunk(int row, int ch) { return (uint32_t)row * 128u + (uint32_t)((ch ^ (row & 7)) << 4); }

// One softmax half of Eq. 6 for one token: u[64] logits in, p[64] (fp32) out in place, its bf16 roundings packed two to a word in pk[32] (what a tensor
// core operand built from p holds).  Returns sum_j bf16(p_j) * vec[j].
template <bool kNeg>
__device__ __forceinline__ float softmax_half_packed(float (&u)[kM], uint32_t (&pk)[kM / 2], const float* vec)
{
    float m = kNeg ? min3(u[0], u[1], u[2]) : max3(u[0], u[1], u[2]);
#pragma unroll
    for (int j = 3; j < kM - 1; j += 2) m = kNeg ? min3(m, u[j], u[j + 1]) : max3(m, u[j], u[j + 1]);
    m = kNeg ? fminf(m, u[kM - 1]) : fmaxf(m, u[kM - 1]);
    const float sL = kNeg ? -kLog2e : kLog2e, off = kNeg ? m * kLog2e : -m * kLog2e;
    const f32x2 scale = pack2(sL, sL), offset = pack2(off, off);
    f32x2 sum2 = pack2(0.f, 0.f);
#pragma unroll
    for (int j = 0; j < kM; j += 2) {
        float x0, x1;
        unpack2(fma2(pack2(u[j], u[j + 1]), scale, offset), x0, x1);
        u[j] = ex2_approx(x0);
        u[j + 1] = ex2_approx(x1);
        sum2 = add2(sum2, pack2(u[j], u[j + 1]));
    }
    float s0, s1;
    unpack2(sum2, s0, s1);
    const float inv = __fdividef(1.f, s0 + s1);
    const f32x2 inv2 = pack2(inv, inv);
    f32x2 dot2 = pack2(0.f, 0.f);
    const float2* vec2 = reinterpret_cast<const float2*>(vec);
#pragma unroll
    for (int j = 0; j < kM; j += 2) {
        unpack2(mul2(pack2(u[j], u[j + 1]), inv2), u[j], u[j + 1]);
        pk[j >> 1] = pack_bf16(u[j], u[j + 1]);
        const float2 zv = vec2[j >> 1];
        dot2 = fma2(pack2(__uint_as_float(pk[j >> 1] << 16), __uint_as_float(pk[j >> 1] & 0xffff0000u)), pack2(zv.x, zv.y), dot2);
    }
    unpack2(dot2, s0, s1);
    return s0 + s1;
}

// The same without roundings and without the division: u[64] becomes e_j = exp(+-u_j - max), `inv_sum` 1 / sum_j e_j
// (p_j = e_j * inv_sum: the callers fold that factor into what they multiply p by); returns sum_j e_j * vec[j].
template <bool kNeg>
__device__ __forceinline__ float softmax_half_raw(float (&u)[kM], float& inv_sum, const float* vec)
{
    float m = kNeg ? min3(u[0], u[1], u[2]) : max3(u[0], u[1], u[2]);
#pragma unroll
    for (int j = 3; j < kM - 1; j += 2) m = kNeg ? min3(m, u[j], u[j + 1]) : max3(m, u[j], u[j + 1]);
    m = kNeg ? fminf(m, u[kM - 1]) : fmaxf(m, u[kM - 1]);
    const float sL = kNeg ? -kLog2e : kLog2e, off = kNeg ? m * kLog2e : -m * kLog2e;
    const f32x2 scale = pack2(sL, sL), offset = pack2(off, off);
    f32x2 sum2 = pack2(0.f, 0.f), dot2 = pack2(0.f, 0.f);
    const float4* vec4 = reinterpret_cast<const float4*>(vec);
#pragma unroll
    for (int j = 0; j < kM; j += 4) {
        const float4 zv = vec4[j >> 2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float x0, x1;
            unpack2(fma2(pack2(u[j + 2 * h], u[j + 2 * h + 1]), scale, offset), x0, x1);
            u[j + 2 * h] = ex2_approx(x0);
            u[j + 2 * h + 1] = ex2_approx(x1);
            const f32x2 e = pack2(u[j + 2 * h], u[j + 2 * h + 1]);
            sum2 = add2(sum2, e);
            dot2 = fma2(e, h ? pack2(zv.z, zv.w) : pack2(zv.x, zv.y), dot2);
        }
    }
    float s0, s1;
    unpack2(sum2, s0, s1);
    inv_sum = __fdividef(1.f, s0 + s1);
    unpack2(dot2, s0, s1);
    return s0 + s1;
}

__device__ __forceinline__ void load64(uint32_t taddr, float (&x)[kM])
{
    uint32_t r[kM];
    tmem_ld_x32(taddr, r);
    tmem_ld_x32(taddr + 32, r + 32);
    tmem_wait_ld();
#pragma unroll
    for (int j = 0; j < kM; ++j) x[j] = __uint_as_float(r[j]);
}

// 64 floats of one token -> bf16 row of a 64-column block (operand / TMA-store layout).
__device__ __forceinline__ void store_row_bf16(uint8_t* blk, int row, const float (&x)[kM])
{
#pragma unroll
    for (int ch = 0; ch < 8; ++ch) {
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) w[q] = pack_bf16(x[8 * ch + 2 * q], x[8 * ch + 2 * q + 1]);
        *reinterpret_cast<uint4*>(blk + sw_chunk(row, ch)) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

// Softmax backward of Eq. 6 for one token, split between the two threads of the token (half 0: softmax(+u),
// half 1: softmax(-u)): each forms p (.) (dphi - p . dphi) for its half; half 1 parks its 64 values in 64 free columns
// of the token's lane of tensor memory (`park`: the columns of T that half 1 itself has just read; both threads of a token
// sit on warps of the same lane quarter, so either can reach the lane), and after a barrier of these warps half 0 takes them back,
// subtracts and writes du (bf16) to its row of the du tile.
__device__ __forceinline__ void du_exchange(int half, int row, const float (&p)[kM], float (&dphi)[kM], uint32_t park, uint8_t* du_tile,
                                            float p_scale = 1.f, float dphi_scale = 1.f)
{
    // the feature values are p_scale * p[], the gradients dphi_scale * dphi[] (the query side keeps the exponentials and
    // their normaliser apart, and the per-token factor 1 / den out of dphi): du_j = a p_j (dphi_j - b sum_i p_i dphi_i) with
    // a = p_scale dphi_scale, b = p_scale
    f32x2 dot2 = pack2(0.f, 0.f);
#pragma unroll
    for (int j = 0; j < kM; j += 2) dot2 = fma2(pack2(p[j], p[j + 1]), pack2(dphi[j], dphi[j + 1]), dot2);
    float d0, d1;
    unpack2(dot2, d0, d1);
    const float as = p_scale * dphi_scale, nd = -(d0 + d1) * p_scale * as;
    const f32x2 ndot = pack2(nd, nd), as2 = pack2(as, as);
#pragma unroll
    for (int j = 0; j < kM; j += 2)
        unpack2(mul2(pack2(p[j], p[j + 1]), fma2(pack2(dphi[j], dphi[j + 1]), as2, ndot)), dphi[j], dphi[j + 1]);
    if (half == 1) {
        uint32_t r[kM];
#pragma unroll
        for (int j = 0; j < kM; ++j) r[j] = __float_as_uint(dphi[j]);
        tmem_st_x32(park, r);
        tmem_st_x32(park + 32, r + 32);
        tmem_wait_st();
    }
    tcgen05_fence_before();
    cbar();
    tcgen05_fence_after();
    if (half == 0) {
        float o[kM];
        load64(park, o);
        const f32x2 minus1 = pack2(-1.f, -1.f);
#pragma unroll
        for (int j = 0; j < kM; j += 2) unpack2(fma2(pack2(o[j], o[j + 1]), minus1, pack2(dphi[j], dphi[j + 1])), dphi[j], dphi[j + 1]);
        store_row_bf16(du_tile, row, dphi);
    }
}

// n products D (+)= A_k B_k issued by one thread, the operands' start addresses advancing by fixed byte steps.  Unrolled,
// so that each descriptor is the first one plus a constant; the first ones pass through `opaque` so that this arithmetic
// stays inside the tile loop (hoisted out of it, the descriptors of a whole tile would not fit the issuer's registers).
__device__ __forceinline__ uint64_t opaque(uint64_t v)
{
    asm volatile("" : "+l"(v));
    return v;
}
template <int kN>
__device__ __forceinline__ void mma_chain_n(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t step_a, uint32_t step_b, uint32_t idesc, uint32_t acc_first)
{
    da = opaque(da);
    db = opaque(db);
#pragma unroll
    for (int k = 0; k < kN; ++k) mma_bf16_ss(d_tmem, da + (uint64_t)(k * (step_a >> 4)), db + (uint64_t)(k * (step_b >> 4)), idesc, k > 0 ? 1u : acc_first);
}
__device__ __forceinline__ void mma_chain(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t step_a, uint32_t step_b, uint32_t idesc, int n,
                                          uint32_t acc_first)
{
    if (n == 4) mma_chain_n<4>(d_tmem, da, db, step_a, step_b, idesc, acc_first);
    else mma_chain_n<8>(d_tmem, da, db, step_a, step_b, idesc, acc_first);
}
// K-major operand tiles are two 64-element blocks of four K steps each (32 bytes apart).
__device__ __forceinline__ uint64_t kmajor_desc() { return make_desc_sw128(0, 16, 1024); }
__device__ __forceinline__ uint64_t mn_desc(uint32_t blk_bytes) { return make_desc_sw128(0, blk_bytes, 1024); }

// U = X W (logits) of one tile: A = X tile, B = W^T image, both K-major.
__device__ __forceinline__ void chain_logits(uint32_t d_tmem, uint32_t x, uint32_t w)
{
    constexpr uint32_t idesc = make_idesc_bf16(kTile, kM, 0, 0);
    mma_chain(d_tmem, desc_at(kmajor_desc(), x), desc_at(kmajor_desc(), w), 32, 32, idesc, 4, 0u);
    mma_chain(d_tmem, desc_at(kmajor_desc(), x + kHalfTileBytes), desc_at(kmajor_desc(), w + kWBytes / 2), 32, 32, idesc, 4, 1u);
}
// T = Y (S_hi + S_lo)^T: A = Y tile (K-major over c), B = image [c][f] read with rows = K (hi pass, then lo pass).
__device__ __forceinline__ void chain_images(uint32_t d_tmem, uint32_t y, uint32_t img_hi, uint32_t img_lo)
{
    constexpr uint32_t idesc = make_idesc_bf16(kTile, kD, 0, 1);
    mma_chain(d_tmem, desc_at(kmajor_desc(), y), desc_at(mn_desc(kHalfTileBytes), img_hi), 32, 2048, idesc, 4, 0u);
    mma_chain(d_tmem, desc_at(kmajor_desc(), y + kHalfTileBytes), desc_at(mn_desc(kHalfTileBytes), img_hi + 4 * 2048), 32, 2048, idesc, 4, 1u);
    mma_chain(d_tmem, desc_at(kmajor_desc(), y), desc_at(mn_desc(kHalfTileBytes), img_lo), 32, 2048, idesc, 4, 1u);
    mma_chain(d_tmem, desc_at(kmajor_desc(), y + kHalfTileBytes), desc_at(mn_desc(kHalfTileBytes), img_lo + 4 * 2048), 32, 2048, idesc, 4, 1u);
}
// dv = phi (dS_hi + dS_lo): A = phi tile (K-major over f), B = image [c][f] read with rows = N (both K-major).
__device__ __forceinline__ void chain_dv(uint32_t d_tmem, uint32_t phi, uint32_t img_hi, uint32_t img_lo)
{
    constexpr uint32_t idesc = make_idesc_bf16(kTile, kD, 0, 0);
    mma_chain(d_tmem, desc_at(kmajor_desc(), phi), desc_at(kmajor_desc(), img_hi), 32, 32, idesc, 4, 0u);
    mma_chain(d_tmem, desc_at(kmajor_desc(), phi + kHalfTileBytes), desc_at(kmajor_desc(), img_hi + kHalfTileBytes), 32, 32, idesc, 4, 1u);
    mma_chain(d_tmem, desc_at(kmajor_desc(), phi), desc_at(kmajor_desc(), img_lo), 32, 32, idesc, 4, 1u);
    mma_chain(d_tmem, desc_at(kmajor_desc(), phi + kHalfTileBytes), desc_at(kmajor_desc(), img_lo + kHalfTileBytes), 32, 32, idesc, 4, 1u);
}
// dS += (phi / den)^T dO: A and B are token tiles read MN-major (K = the tile's tokens).
__device__ __forceinline__ void chain_ds(uint32_t d_tmem, uint32_t phi, uint32_t g, bool first_of_segment)
{
    constexpr uint32_t idesc = make_idesc_bf16(kD, kD, 1, 1);
    mma_chain(d_tmem, desc_at(mn_desc(kHalfTileBytes), phi), desc_at(mn_desc(kHalfTileBytes), g), 2048, 2048, idesc, kTile / 16, first_of_segment ? 0u : 1u);
}
// dx = du W^T and dW += x^T du for one tile: A of the first product is the du tile (K-major, K = 64), B the W^T image
// [j][c] read MN-major; the second product reads the x tile MN-major (x^T) and du MN-major.
__device__ __forceinline__ void chain_dx_dw(uint32_t t_dx, uint32_t t_dw, uint32_t du, uint32_t x, uint32_t w, bool first_of_segment)
{
    constexpr uint32_t idesc_dx = make_idesc_bf16(kTile, kD, 0, 1);
    constexpr uint32_t idesc_dw = make_idesc_bf16(kD, kM, 1, 1);
    mma_chain(t_dx, desc_at(kmajor_desc(), du), desc_at(mn_desc(kWBytes / 2), w), 32, 2048, idesc_dx, kM / 16, 0u);
    mma_chain(t_dw, desc_at(mn_desc(kHalfTileBytes), x), desc_at(mn_desc(kHalfTileBytes), du), 2048, 2048, idesc_dw, kTile / 16, first_of_segment ? 0u : 1u);
}

// Write the weight-gradient accumulator (TMEM: lane = input feature c, 64 columns = logits j) as a [j][c] record.
__device__ __forceinline__ void drain_dw(uint32_t t_dw, uint32_t lane_base, int half, int row, float* rec)
{
    uint32_t v[32];
    tmem_ld_x32(t_dw + lane_base + half * 32, v);
    tmem_wait_ld();
#pragma unroll
    for (int j = 0; j < 32; ++j) rec[(size_t)(half * 32 + j) * kD + row] = __uint_as_float(v[j]);
}

// Unwinding after a wait that gave up: whatever copies into shared memory are still in flight (requested by this warp or
// by the store warp, which requests none after the two have met) get a short while to land before the CTA gives its shared
// memory back.  A barrier whose current phase has no copy outstanding just runs out the short limit.
__device__ __forceinline__ void settle_copies(const BwdCta& c, uint32_t ph_seg, uint32_t ph_x0, uint32_t ph_x1, uint32_t ph_in2)
{
    constexpr uint64_t kSettleNs = 20000;
    mbar_wait(c.bar(BW_SEG), ph_seg, kSettleNs);
    mbar_wait(c.bar(BW_X0), ph_x0, kSettleNs);
    mbar_wait(c.bar(BW_X1), ph_x1, kSettleNs);
    mbar_wait(c.bar(BW_IN2), ph_in2, kSettleNs);
}

// The issuer's and the store warp's waits: the whole warp waits (bounded), the verdict is warp-uniform.
__device__ __forceinline__ bool issuer_wait(const BwdCta& c, int b, uint32_t& phase, uint32_t code)
{
    const bool ok = warp_wait(c.bar(b), phase, c.wc, code);
    phase ^= 1u;
    tcgen05_fence_after();
    return ok;
}

// Schedule of a head's tiles, both kernels (i = tile):
//   issuer:        wait OPS(i) | logits(i+1), last stage(i) | copies into the buffers that stage frees | T(i+1) |
//                  wait STAGED(i), stores of tile i, PFREE
//   element-wise:  feature map(i+1) | wait GFULL(i), results of tile i to their staging tiles, STAGED(i) |
//                  wait TFULL(i+1), ... du(i+1), operands of the last stage written, OPS(i+1)
// so the tensor core works on tile i's last stage and tile i+1's first products while the CUDA cores run tile i+1's
// feature map and convert tile i's results.  The first tile of a head starts from scratch (images and weights change
// there) and the last one is finished before the next head's copies are requested.
template <int kLayout, int kMixB>
__global__ void __launch_bounds__(kBwdThreads, 1)
qside_bwd_tc(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmG,
             const __grid_constant__ CUtensorMap tmDQ, const __grid_constant__ CUtensorMap tmW,
             const __grid_constant__ CUtensorMap tmShi, const __grid_constant__ CUtensorMap tmSlo, const BwdArgs a)
{
    extern __shared__ uint8_t bwd_smem[];
    using L = BwdSmemQ;
    if (!bwd_smem_fits(bwd_smem, kBwdSmemQ, a.err)) return;
    const BwdCta c = bwd_setup(bwd_smem, L::kMisc, a.err, a.wait_limit_us);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // tensor memory: logits | T = dO S^T (later the du exchange) | dS | dW_q | dq
    const uint32_t t_u = c.tmem, t_t = c.tmem + 64, t_ds = c.tmem + 192, t_dw = c.tmem + 320, t_dq = c.tmem + 384;
    const uint32_t sb0 = c.sbase;
    TileWalk w;
    w.init(a.total_tiles, a.tiles_per_head);

    if (warp >= kBwdIssuer) {
        setmaxnreg_dec<kBwdRegsIssuer>();
        if (warp <= kBwdIssuer + 1) {
            // =================== issuer (warp 8) and store warp (warp 9) ===================
            const bool one = lane == 0;
            if (one) {
                tma_prefetch_desc(&tmQ);
                tma_prefetch_desc(&tmG);
                tma_prefetch_desc(&tmDQ);
            }
            auto xbuf = [&](int b) { return sb0 + (b ? L::kX1 : L::kX0); };
            auto load_seg = [&](const TileWalk& t) {   // S (hi, lo) and W_q^T of the head
                mbar_arrive_expect_tx(c.bar(BW_SEG), 2 * kTileBytes + kWBytes);
                for (int b = 0; b < 2; ++b) {
                    tma_load_3d(sb0 + L::kShi + b * kHalfTileBytes, &tmShi, c.bar(BW_SEG), 64 * b, 0, t.g);
                    tma_load_3d(sb0 + L::kSlo + b * kHalfTileBytes, &tmSlo, c.bar(BW_SEG), 64 * b, 0, t.g);
                    tma_load_3d(sb0 + L::kW + b * (kWBytes / 2), &tmW, c.bar(BW_SEG), 64 * b, 0, t.g % a.H);
                }
            };
            auto load_q = [&](const TileWalk& t, int buf) {
                mbar_arrive_expect_tx(c.bar(BW_X0 + buf), kTileBytes);
                for (int b = 0; b < 2; ++b) act_load<kLayout>(xbuf(buf) + b * kHalfTileBytes, &tmQ, c.bar(BW_X0 + buf), 64 * b, t.lt * kTile, t.g, a.H);
            };
            auto load_g = [&](const TileWalk& t) {   // dO; the tile after it starts on its way into L2
                mbar_arrive_expect_tx(c.bar(BW_IN2), kTileBytes);
                for (int b = 0; b < 2; ++b) act_load<kLayout>(sb0 + L::kG + b * kHalfTileBytes, &tmG, c.bar(BW_IN2), 64 * b, t.lt * kTile, t.g, a.H);
                TileWalk n2 = t;
                n2.next();
                if (!n2.done())
                    for (int b = 0; b < 2; ++b) act_prefetch_l2<kLayout>(&tmG, 64 * b, n2.lt * kTile, n2.g, a.H);
            };
            auto issue_t = [&]() {   // T = dO S^T (S_hi, S_lo)
                chain_images(t_t, sb0 + L::kG, sb0 + L::kShi, sb0 + L::kSlo);
                mma_commit(c.bar(BW_TFULL));
            };
            if (warp == kBwdIssuer + 1) {
                // =================== store warp ===================
                uint32_t ph_staged = 0;
                int xb = 0;
                for (; !w.done(); w.next(), xb ^= 1) {
                    const bool last = w.last();
                    TileWalk nx = w;
                    nx.next();
                    TileWalk nn = nx;
                    nn.next();
                    const bool ahead = !last && !nx.done();
                    const bool ahead2 = ahead && !nx.last() && !nn.done();
                    // dq of this tile has been staged in the tile's own Q buffer (so its last stage is complete): store it; the
                    // buffer then takes the Q of the tile after the next, or, at the end of a head, everything is free for
                    // the next head's copies
                    if (!issuer_wait(c, BW_STAGED, ph_staged, kErrStore)) break;
                    if (one) {
                        for (int b = 0; b < 2; ++b) act_store<kLayout>(&tmDQ, xbuf(xb) + b * kHalfTileBytes, 64 * b, w.lt * kTile, w.g, a.H);
                        bulk_commit_group();
                        if (ahead2) {
                            bulk_wait_group_read<0>();
                            load_q(nn, xb);
                        } else if (!ahead && !nx.done()) {
                            bulk_wait_group_read<0>();   // (the store before this one read the other Q buffer)
                            load_seg(nx);
                            load_q(nx, xb ^ 1);
                            load_g(nx);
                        }
                    }
                    __syncwarp();
                }
                if (one) bulk_wait_group<0>();
                named_barrier_sync(2, 64);   // no copy is requested after this point
            } else {
            // =================== issuer ===================
            uint32_t ph_x[2] = {0u, 0u}, ph_in2 = 0, ph_seg = 0, ph_ops1 = 0, ph_ops = 0, ph_g1 = 0;
            bool ok = true, pre = false;
            int xb = 0;
            if (!w.done() && one) {
                load_seg(w);
                load_q(w, 0);
                load_g(w);
            }
            for (; !w.done(); w.next(), xb ^= 1) {
                const bool first = w.first(), last = w.last();
                TileWalk nx = w;
                nx.next();
                const bool ahead = !last && !nx.done();   // the next tile belongs to the same head
                if (!pre) {
                    // ---- the head's first tile: U = Q W_q once Q, W_q are there, T = dO S^T once dO, S are there ----
                    if (first) {
                        if (!issuer_wait(c, BW_SEG, ph_seg, kErrSeg)) { ok = false; break; }
                    }
                    if (!issuer_wait(c, BW_X0 + xb, ph_x[xb], kErrMmaLoad)) { ok = false; break; }
                    if (one) {
                        chain_logits(t_u, xbuf(xb), sb0 + L::kW);
                        mma_commit(c.bar(BW_LFULL));
                        if (ahead) load_q(nx, xb ^ 1);
                    }
                    if (!issuer_wait(c, BW_IN2, ph_in2, kErrMmaLoad)) { ok = false; break; }
                    if (one) issue_t();
                    __syncwarp();
                }
                // ---- phi / den of this tile is written: dS += (phi / den)^T dO at once, so that dO's tile is free for the
                // next tile's dO while this tile's du is still being formed ----
                if (!issuer_wait(c, BW_OPS1, ph_ops1, kErrMmaPhi)) { ok = false; break; }
                LB_TRACE_I(2, 0);
                if (one) {
                    chain_ds(t_ds, sb0 + L::kP, sb0 + L::kG, first);
                    mma_commit(c.bar(BW_G1));
                }
                __syncwarp();
                LB_TRACE_I(2, 1);
                if (ahead) {
                    // the next tile's logits (this tile's have long been read, and its Q came in a tile ago)
                    if (!issuer_wait(c, BW_X0 + (xb ^ 1), ph_x[xb ^ 1], kErrMmaLoad)) { ok = false; break; }
                    if (one) {
                        chain_logits(t_u, xbuf(xb ^ 1), sb0 + L::kW);
                        mma_commit(c.bar(BW_LFULL));
                    }
                    __syncwarp();
                }
                LB_TRACE_I(2, 2);
                if (!issuer_wait(c, BW_G1, ph_g1, kErrMmaAcc)) { ok = false; break; }
                LB_TRACE_I(2, 3);
                if (ahead && one) load_g(nx);
                // ---- du is written: dq = du W_q^T, dW_q += Q^T du, then the next tile's T = dO S^T (the element-wise warps
                // took this tile's T out of tensor memory before they announced phi / den, and are done with the columns
                // they exchange du through) ----
                if (!issuer_wait(c, BW_OPS, ph_ops, kErrMmaPhi)) { ok = false; break; }
                LB_TRACE_I(2, 4);
                if (one) {
                    chain_dx_dw(t_dq, t_dw, sb0 + L::kDu, xbuf(xb), sb0 + L::kW, first);
                    mma_commit(c.bar(BW_GFULL));
                }
                __syncwarp();
                LB_TRACE_I(2, 5);
                if (ahead) {
                    if (!issuer_wait(c, BW_IN2, ph_in2, kErrMmaLoad)) { ok = false; break; }
                    LB_TRACE_I(2, 6);
                    if (one) issue_t();
                    __syncwarp();
                    LB_TRACE_I(2, 7);
                }
                pre = ahead;
            }
            named_barrier_sync(2, 64);
            if (!ok) settle_copies(c, ph_seg, ph_x[0], ph_x[1], ph_in2);
            }
        }
    } else {
        setmaxnreg_inc<kBwdRegsCompute>();
        // =================== element-wise warps ===================
        const int half = warp >> 2, row = (warp & 3) * 32 + lane;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        float* vec = c.misc + BwdMisc::kVec / 4;
        float* sa = c.misc + BwdMisc::kA / 4;
        float* sb = c.misc + BwdMisc::kB / 4;
        float* sdd = sb;   // dden den of the tile's tokens takes the place of the first half of sb once both halves have been read
        uint32_t ph_l = 0, ph_t = 0, ph_g = 0;
        float dr_acc = 0.f;   // Eq. 8: this thread's share of sum dout . (a - o)
        f32x2 dz2[4];         // thread (8 consecutive features as 4 pairs, 8 of the tile's tokens); summed over the token groups at the end of a segment
#pragma unroll
        for (int e = 0; e < 4; ++e) dz2[e] = pack2(0.f, 0.f);
        // dq of a tile leaves tensor memory for the tile's own Q buffer (the tile's last tensor-core stage has completed)
        auto stage_dq = [&](int buf) {
            float x[kM];
            load64(t_dq + lane_base + half * kM, x);
            store_row_bf16(c.smem + (buf ? L::kX1 : L::kX0) + half * kHalfTileBytes, row, x);
            warp_announce(c, BW_STAGED);
        };
        bool pre = false;   // the previous tile belongs to the same head: its dq is still in tensor memory
        int xb = 0;
        for (; !w.done(); w.next(), xb ^= 1) {
            const bool first = w.first(), last = w.last();
            TileWalk nx = w;
            nx.next();
            LB_TRACE(0);
            if (first && tid < kD) vec[tid] = a.state[(size_t)w.g * kE + kD * kD + tid];   // z (read after the next barrier)
            bool okl = wait_only(c, BW_LFULL, ph_l, kErrSoftmaxU);   // verdict of this warp's waits since the last barrier with a verdict
            LB_TRACE(2);
            if (first && !cbar_and(okl)) break;
            // ---- phi(q): p stays in registers (fp32, and its bf16 roundings); den = phi . z from the rounded values ----
            float p[kM];
            load64(t_u + lane_base, p);
            float invs;   // p_j = invs * p[j] from here on
            {
                const float ez = half == 0 ? softmax_half_raw<false>(p, invs, vec) : softmax_half_raw<true>(p, invs, vec + kM);
                sa[half * kTile + row] = ez * invs;
            }
            LB_TRACE(3);
            if (pre) {
                // ---- the previous tile's last stage has had the time of a feature map: its dq leaves ----
                if (!compute_wait(c, BW_GFULL, ph_g, kErrStore, okl)) break;
                LB_TRACE(6);
                stage_dq(xb ^ 1);
                LB_TRACE(7);
            }
            if (!compute_wait(c, BW_TFULL, ph_t, kErrEpilogue, okl)) break;   // T is there (and every thread's den part is visible)
            LB_TRACE(4);
            // ---- dO . o = (dO S^T) . phi / den: the numerator phi S itself is never formed.  The per-token factor 1 / den of
            // dnum = dO / den is kept OUT of the tensor-core operands: dphi = (dO S^T - (dO . o) z) / den is scaled here, in
            // the accumulator's epilogue, and dS = (phi / den)^T dO takes it into phi, so the dO tile itself, exact in bf16,
            // is the operand of both products ----
            float x[kM];
            load64(t_t + lane_base + half * kM, x);
            const float inv1 = 1.f / (sa[row] + sa[kTile + row]);
            const float inv = inv1 * a.lin_scale;   // every gradient below is linear in the incoming one: its factor rides on 1 / den
            {
                f32x2 gs2 = pack2(0.f, 0.f);
#pragma unroll
                for (int j = 0; j < kM; j += 2)
                    gs2 = fma2(pack2(p[j], p[j + 1]), pack2(x[j], x[j + 1]), gs2);
                float g0s, g1s;
                unpack2(gs2, g0s, g1s);
                g0s *= invs;
                g1s *= invs;
                sb[half * kTile + row] = (g0s + g1s) * inv1;   // this half's part of dO . o
                if (kMixB) {
                    // Eq. 8: dout . a over this thread's 64 columns (dout from its tile, a straight from memory: one
                    // 128-byte line per thread, started towards L2 a tile ago), minus this half's part of dout . o
                    dr_acc -= (g0s + g1s) * inv1;
                    const int token = w.lt * kTile + row;
                    if (token < a.n) {
                        const __nv_bfloat16* ap = a.mix_a + (size_t)(w.g / a.H) * a.str_batch + (size_t)(w.g % a.H) * a.str_head +
                                                  (size_t)token * a.str_token + half * kM;
                        const uint8_t* gblk = c.smem + L::kG + half * kHalfTileBytes;
                        f32x2 da2 = pack2(0.f, 0.f);
#pragma unroll
                        for (int ch = 0; ch < 8; ++ch) {
                            const uint4 av = __ldg(reinterpret_cast<const uint4*>(ap) + ch);
                            const uint4 gv = *reinterpret_cast<const uint4*>(gblk + sw_chunk(row, ch));
                            const uint32_t aw[4] = {av.x, av.y, av.z, av.w}, gw[4] = {gv.x, gv.y, gv.z, gv.w};
#pragma unroll
                            for (int q = 0; q < 4; ++q)
                                da2 = fma2(pack2(__uint_as_float(gw[q] << 16), __uint_as_float(gw[q] & 0xffff0000u)),
                                           pack2(__uint_as_float(aw[q] << 16), __uint_as_float(aw[q] & 0xffff0000u)), da2);
                        }
                        float d0, d1;
                        unpack2(da2, d0, d1);
                        dr_acc += d0 + d1;
                    }
                    if (!nx.done() && nx.lt * kTile + row < a.n)
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(a.mix_a + (size_t)(nx.g / a.H) * a.str_batch + (size_t)(nx.g % a.H) * a.str_head +
                                                                     (size_t)(nx.lt * kTile + row) * a.str_token + half * kM));
                }
                // phi / den (bf16) is the operand of dS and the factor of dz (the previous tile's dS and dz are done with the tile)
                float y[kM];
                const f32x2 inv2 = pack2(inv * invs, inv * invs);
#pragma unroll
                for (int j = 0; j < kM; j += 2) unpack2(mul2(pack2(p[j], p[j + 1]), inv2), y[j], y[j + 1]);
                store_row_bf16(c.smem + L::kP + half * kHalfTileBytes, row, y);
                warp_announce(c, BW_OPS1);
            }
            cbar();
            const float ngo = -(sb[row] + sb[kTile + row]);   // -(dO . o) = dden * den
            LB_TRACE(5);
            // ---- du (through the softmax of Eq. 6) ----
#pragma unroll
            for (int j = 0; j < kM; j += 4) {   // dphi = (dO S^T - (dO . o) z) / den, its factor 1 / den left to the next step
                const float4 zv = *reinterpret_cast<const float4*>(&vec[half * kM + j]);
                unpack2(fma2(pack2(ngo, ngo), pack2(zv.x, zv.y), pack2(x[j], x[j + 1])), x[j], x[j + 1]);
                unpack2(fma2(pack2(ngo, ngo), pack2(zv.z, zv.w), pack2(x[j + 2], x[j + 3])), x[j + 2], x[j + 3]);
            }
            du_exchange(half, row, p, x, t_t + kM + lane_base, c.smem + L::kDu, invs, inv);   // (a barrier inside: both halves of sb have been read)
            if (half == 0) sdd[row] = ngo;
            if (!(a.test_unmet && warp == 0 && w.i == 0)) warp_announce(c, BW_OPS);   // (left out once by the test of the time-out path)
            cbar();
            LB_TRACE(8);
            {
                // dz += phi^T dden = (phi / den)^T (dden den) on the CUDA cores: thread = (16-byte chunk of 8 features,
                // group of 8 tokens)
                const int fc = tid & 15, t0 = (tid >> 4) * 8;
                const uint8_t* blk = c.smem + L::kP + (fc >> 3) * kHalfTileBytes;
#pragma unroll
                for (int t = t0; t < t0 + 8; ++t) {
                    const uint4 pv = *reinterpret_cast<const uint4*>(blk + sw_chunk(t, fc & 7));
                    const uint32_t pw[4] = {pv.x, pv.y, pv.z, pv.w};
                    const float dd = sdd[t];
                    const f32x2 dd2 = pack2(dd, dd);
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        dz2[q] = fma2(dd2, pack2(__uint_as_float(pw[q] << 16), __uint_as_float(pw[q] & 0xffff0000u)), dz2[q]);
                }
            }
            LB_TRACE(9);
            pre = !last && !nx.done();
            if (pre) continue;

            // ---- the last tile of the head (or of the run): finished here; the accumulators go to the (CTA, head) records ----
            if (!compute_wait(c, BW_GFULL, ph_g, kErrStore)) break;
            stage_dq(xb);
            {
                float* rec = a.part_state + (size_t)(blockIdx.x + w.g) * kE;
                {
                    float x[kM];
                    load64(t_ds + lane_base + half * kM, x);   // lane = feature f, columns = c
#pragma unroll
                    for (int j = 0; j < kM; ++j) rec[(size_t)(half * kM + j) * kD + row] = x[j];
                }
                drain_dw(t_dw, lane_base, half, row, a.part_w + (size_t)(blockIdx.x + w.g) * kWRec);
                // dz: the 16 token groups' sums, in group order (the du tile has been consumed)
                float* red = reinterpret_cast<float*>(c.smem + L::kRed);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float d0, d1;
                    unpack2(dz2[e], d0, d1);
                    red[(tid >> 4) * kD + (tid & 15) * 8 + 2 * e] = d0;
                    red[(tid >> 4) * kD + (tid & 15) * 8 + 2 * e + 1] = d1;
                    dz2[e] = pack2(0.f, 0.f);
                }
                cbar();
                if (tid < kD) {
                    float acc = 0.f;
#pragma unroll
                    for (int gidx = 0; gidx < 16; ++gidx) acc += red[gidx * kD + tid];
                    rec[kD * kD + tid] = acc;
                }
            }
            tcgen05_fence_before();
            cbar();
            LB_TRACE(11);
        }
        if (kMixB) {
            // the CTA's sum of dout . (a - o), thread by thread in index order (bit-reproducible)
            float* red = reinterpret_cast<float*>(c.smem + L::kRed);
            cbar();
            red[tid] = dr_acc;
            cbar();
            if (tid == 0) {
                float acc = 0.f;
                for (int i = 0; i < kBwdCompute; ++i) acc += red[i];
                a.part_dr[blockIdx.x] = acc;
            }
        }
    }
    bwd_teardown(c);
}

template <int kLayout>
__global__ void __launch_bounds__(kBwdThreads, 1)
kside_bwd_tc(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
             const __grid_constant__ CUtensorMap tmDK, const __grid_constant__ CUtensorMap tmDV,
             const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmShi,
             const __grid_constant__ CUtensorMap tmSlo, const BwdArgs a)
{
    extern __shared__ uint8_t bwd_smem[];
    using L = BwdSmemK;
    if (!bwd_smem_fits(bwd_smem, kBwdSmemK, a.err)) return;
    const BwdCta c = bwd_setup(bwd_smem, L::kMisc, a.err, a.wait_limit_us);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // tensor memory: logits | T = V dS^T (later the du exchange) | dv | dW_k | dk
    const uint32_t t_u = c.tmem, t_t = c.tmem + 64, t_dv = c.tmem + 192, t_dw = c.tmem + 320, t_dk = c.tmem + 384;
    const uint32_t sb0 = c.sbase;
    TileWalk w;
    w.init(a.total_tiles, a.tiles_per_head);

    if (warp >= kBwdIssuer) {
        setmaxnreg_dec<kBwdRegsIssuer>();
        if (warp <= kBwdIssuer + 1) {
            // =================== issuer (warp 8) and store warp (warp 9) ===================
            const bool one = lane == 0;
            if (one) {
                tma_prefetch_desc(&tmK);
                tma_prefetch_desc(&tmV);
                tma_prefetch_desc(&tmDK);
                tma_prefetch_desc(&tmDV);
            }
            auto xbuf = [&](int b) { return sb0 + (b ? L::kX1 : L::kX0); };
            auto load_seg = [&](const TileWalk& t) {   // dS (hi, lo) and W_k^T of the head
                mbar_arrive_expect_tx(c.bar(BW_SEG), 2 * kTileBytes + kWBytes);
                for (int b = 0; b < 2; ++b) {
                    tma_load_3d(sb0 + L::kShi + b * kHalfTileBytes, &tmShi, c.bar(BW_SEG), 64 * b, 0, t.g);
                    tma_load_3d(sb0 + L::kSlo + b * kHalfTileBytes, &tmSlo, c.bar(BW_SEG), 64 * b, 0, t.g);
                    tma_load_3d(sb0 + L::kW + b * (kWBytes / 2), &tmW, c.bar(BW_SEG), 64 * b, 0, t.g % a.H);
                }
            };
            auto load_k = [&](const TileWalk& t, int buf) {
                mbar_arrive_expect_tx(c.bar(BW_X0 + buf), kTileBytes);
                for (int b = 0; b < 2; ++b) act_load<kLayout>(xbuf(buf) + b * kHalfTileBytes, &tmK, c.bar(BW_X0 + buf), 64 * b, t.lt * kTile, t.g, a.H);
                TileWalk n2 = t;
                n2.next();
                if (!n2.done())
                    for (int b = 0; b < 2; ++b) act_prefetch_l2<kLayout>(&tmK, 64 * b, n2.lt * kTile, n2.g, a.H);
            };
            auto load_v = [&](const TileWalk& t) {
                mbar_arrive_expect_tx(c.bar(BW_IN2), kTileBytes);
                for (int b = 0; b < 2; ++b) act_load<kLayout>(sb0 + L::kV + b * kHalfTileBytes, &tmV, c.bar(BW_IN2), 64 * b, t.lt * kTile, t.g, a.H);
                TileWalk n2 = t;
                n2.next();
                if (!n2.done())
                    for (int b = 0; b < 2; ++b) act_prefetch_l2<kLayout>(&tmV, 64 * b, n2.lt * kTile, n2.g, a.H);
            };
            auto issue_t = [&]() {   // T = V dS^T (hi and lo parts of dS)
                chain_images(t_t, sb0 + L::kV, sb0 + L::kShi, sb0 + L::kSlo);
                mma_commit(c.bar(BW_TFULL));
            };
            if (warp == kBwdIssuer + 1) {
                // =================== store warp ===================
                uint32_t ph_staged1 = 0, ph_staged = 0;
                int xb = 0;
                for (; !w.done(); w.next(), xb ^= 1) {
                    const bool last = w.last();
                    TileWalk nx = w;
                    nx.next();
                    TileWalk nn = nx;
                    nn.next();
                    const bool ahead = !last && !nx.done();
                    const bool ahead2 = ahead && !nx.last() && !nn.done();
                    // dk has been staged in this tile's K buffer (dk and dW_k are complete): store it; the buffer then takes the
                    // K of the tile after the next
                    if (!issuer_wait(c, BW_STAGED1, ph_staged1, kErrStore)) break;
                    if (one) {
                        for (int b = 0; b < 2; ++b) act_store<kLayout>(&tmDK, xbuf(xb) + b * kHalfTileBytes, 64 * b, w.lt * kTile, w.g, a.H);
                        bulk_commit_group();
                        if (ahead2) {
                            bulk_wait_group_read<0>();
                            load_k(nn, xb);
                        }
                    }
                    __syncwarp();
                    // dv has been staged in V's tile (the next tile's V dS^T is done with it): store it; the tile then takes the V
                    // of the tile after the next, or, at the end of a head, everything is free for the next head's copies
                    if (!issuer_wait(c, BW_STAGED, ph_staged, kErrStore)) break;
                    if (one) {
                        for (int b = 0; b < 2; ++b) act_store<kLayout>(&tmDV, sb0 + L::kV + b * kHalfTileBytes, 64 * b, w.lt * kTile, w.g, a.H);
                        bulk_commit_group();
                        if (ahead2) {
                            bulk_wait_group_read<0>();
                            load_v(nn);
                        } else if (!ahead && !nx.done()) {
                            bulk_wait_group_read<0>();
                            load_seg(nx);
                            load_k(nx, xb ^ 1);
                            load_v(nx);
                        }
                    }
                    __syncwarp();
                }
                if (one) bulk_wait_group<0>();
                named_barrier_sync(2, 64);   // no copy is requested after this point
            } else {
            // =================== issuer ===================
            uint32_t ph_x[2] = {0u, 0u}, ph_in2 = 0, ph_seg = 0, ph_ops1 = 0, ph_ops = 0, ph_t = 0;
            bool ok = true, pre = false;
            int xb = 0;
            if (!w.done() && one) {
                load_seg(w);
                load_k(w, 0);
                load_v(w);
            }
            for (; !w.done(); w.next(), xb ^= 1) {
                const bool first = w.first(), last = w.last();
                TileWalk nx = w;
                nx.next();
                const bool ahead = !last && !nx.done();
                if (!pre) {
                    // ---- the head's first tile: U = K W_k once K, W_k are there, T = V dS^T once V, dS are there; V's tile then
                    // takes the next tile's V ----
                    if (first) {
                        if (!issuer_wait(c, BW_SEG, ph_seg, kErrSeg)) { ok = false; break; }
                    }
                    if (!issuer_wait(c, BW_X0 + xb, ph_x[xb], kErrMmaLoad)) { ok = false; break; }
                    if (one) {
                        chain_logits(t_u, xbuf(xb), sb0 + L::kW);
                        mma_commit(c.bar(BW_LFULL));
                        if (ahead) load_k(nx, xb ^ 1);
                    }
                    if (!issuer_wait(c, BW_IN2, ph_in2, kErrMmaLoad)) { ok = false; break; }
                    if (one) issue_t();
                    __syncwarp();
                    if (ahead) {
                        if (!issuer_wait(c, BW_TFULL, ph_t, kErrMmaAcc)) { ok = false; break; }
                        if (one) load_v(nx);
                    } else {
                        ph_t ^= 1u;   // (that phase is not waited for here)
                    }
                } else {
                    ph_t ^= 1u;       // this tile's V dS^T was issued during the previous tile
                }
                // ---- this tile's logits have been read: the next tile's; then, phi and du of this tile written,
                // dk = du W_k^T and dW_k += K^T du (the du tile and this tile's K buffer are free after them), the next
                // tile's V dS^T, and dv = phi dS (hi and lo parts) last ----
                if (!issuer_wait(c, BW_OPS1, ph_ops1, kErrMmaU)) { ok = false; break; }
                LB_TRACE_I(3, 0);
                if (ahead) {
                    if (!issuer_wait(c, BW_X0 + (xb ^ 1), ph_x[xb ^ 1], kErrMmaLoad)) { ok = false; break; }
                    if (one) {
                        chain_logits(t_u, xbuf(xb ^ 1), sb0 + L::kW);
                        mma_commit(c.bar(BW_LFULL));
                    }
                    __syncwarp();
                }
                LB_TRACE_I(3, 1);
                if (!issuer_wait(c, BW_OPS, ph_ops, kErrMmaPhi)) { ok = false; break; }
                LB_TRACE_I(3, 2);
                if (one) {
                    chain_dx_dw(t_dk, t_dw, sb0 + L::kDu, xbuf(xb), sb0 + L::kW, first);
                    mma_commit(c.bar(BW_G1));
                }
                __syncwarp();
                LB_TRACE_I(3, 3);
                if (ahead) {
                    if (!issuer_wait(c, BW_IN2, ph_in2, kErrMmaLoad)) { ok = false; break; }
                    LB_TRACE_I(3, 4);
                    if (one) issue_t();   // the element-wise warps took this tile's T out of tensor memory before they announced its operands
                }
                __syncwarp();
                LB_TRACE_I(3, 5);
                if (one) {
                    chain_dv(t_dv, sb0 + L::kP, sb0 + L::kShi, sb0 + L::kSlo);
                    mma_commit(c.bar(BW_GFULL));
                }
                __syncwarp();
                LB_TRACE_I(3, 6);
                pre = ahead;
            }
            named_barrier_sync(2, 64);
            if (!ok) settle_copies(c, ph_seg, ph_x[0], ph_x[1], ph_in2);
            }
        }
    } else {
        setmaxnreg_inc<kBwdRegsCompute>();
        // =================== element-wise warps ===================
        const int half = warp >> 2, row = (warp & 3) * 32 + lane;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        float* vec = c.misc + BwdMisc::kVec / 4;
        uint32_t ph_l = 0, ph_t = 0, ph_g1 = 0, ph_g = 0;
        // dk of a tile leaves tensor memory for the tile's own K buffer (dk and dW_k are complete: the buffer has been read)
        auto stage_dk = [&](int buf) {
            float x[kM];
            load64(t_dk + lane_base + half * kM, x);
            store_row_bf16(c.smem + (buf ? L::kX1 : L::kX0) + half * kHalfTileBytes, row, x);
            warp_announce(c, BW_STAGED1);
        };
        // dv leaves for V's tile (the V dS^T that read it last is complete)
        auto stage_dv = [&]() {
            float x[kM];
            load64(t_dv + lane_base + half * kM, x);
            store_row_bf16(c.smem + L::kV + half * kHalfTileBytes, row, x);
            warp_announce(c, BW_STAGED);
        };
        bool pre = false;
        bool okl = true;   // verdict of this warp's waits since the last barrier with a verdict (a warp leaves only at such a barrier)
        int xb = 0;
        for (; !w.done(); w.next(), xb ^= 1) {
            const bool first = w.first(), last = w.last();
            TileWalk nx = w;
            nx.next();
            LB_TRACE_K(0);
            if (first && tid < kD) vec[tid] = a.state[(size_t)w.g * kE + kD * kD + tid];   // dz (read after the next barrier)
            okl = wait_only(c, BW_LFULL, ph_l, kErrSoftmaxU) && okl;
            LB_TRACE_K(2);
            // ---- phi(k): p stays in registers (fp32, and its bf16 roundings, which go to phi's tile once that is free) ----
            float p[kM];
            uint32_t pk[kM / 2];
            load64(t_u + lane_base, p);
            warp_announce(c, BW_OPS1);   // the logits' columns may take the next tile's
            if (half == 0) softmax_half_packed<false>(p, pk, vec);   // (the returned dot product is not needed here: vec may still be the old one)
            else softmax_half_packed<true>(p, pk, vec + kM);
            LB_TRACE_K(3);
            if (pre) {
                // ---- the previous tile's dk and dW_k have had the time of a feature map: dk leaves, the du tile is free ----
                if (!compute_wait(c, BW_G1, ph_g1, kErrStore, okl)) break;
                LB_TRACE_K(6);
                stage_dk(xb ^ 1);
                LB_TRACE_K(7);
            }
            if (!compute_wait(c, BW_TFULL, ph_t, kErrMmaAcc, okl)) break;
            LB_TRACE_K(4);
            // ---- dphi = V dS^T + dz -> du ----
            {
                float x[kM];
                load64(t_t + lane_base + half * kM, x);
#pragma unroll
                for (int j = 0; j < kM; j += 2) {
                    const float2 zv = *reinterpret_cast<const float2*>(&vec[half * kM + j]);
                    unpack2(add2(pack2(x[j], x[j + 1]), pack2(zv.x, zv.y)), x[j], x[j + 1]);
                }
                du_exchange(half, row, p, x, t_t + kM + lane_base, c.smem + L::kDu);
            }
            LB_TRACE_K(5);
            if (pre) {
                // ---- the previous tile's dv is complete: it leaves through V's tile, and phi's tile is free ----
                if (!compute_wait(c, BW_GFULL, ph_g, kErrStore)) break;
                LB_TRACE_K(10);
                stage_dv();
                LB_TRACE_K(11);
            }
            {
                uint8_t* blk = c.smem + L::kP + half * kHalfTileBytes;
#pragma unroll
                for (int ch = 0; ch < 8; ++ch)
                    *reinterpret_cast<uint4*>(blk + sw_chunk(row, ch)) = make_uint4(pk[4 * ch], pk[4 * ch + 1], pk[4 * ch + 2], pk[4 * ch + 3]);
            }
            if (!(a.test_unmet && warp == 0 && w.i == 0)) warp_announce(c, BW_OPS);   // (left out once by the test of the time-out path)
            LB_TRACE_K(8);
            pre = !last && !nx.done();
            if (pre) continue;
            // ---- the last tile of the head (or of the run): finished here ----
            if (!compute_wait(c, BW_G1, ph_g1, kErrStore)) break;
            stage_dk(xb);
            if (!compute_wait(c, BW_GFULL, ph_g, kErrStore)) break;
            stage_dv();
            drain_dw(t_dw, lane_base, half, row, a.part_w + (size_t)(blockIdx.x + w.g) * kWRec);
            tcgen05_fence_before();
            cbar();
        }
    }
    bwd_teardown(c);
}

// out[g][e] = sum over the CTAs that own tiles of head g, ascending, of part[(cta + g)][e].  grid = (ceil(E/256), G).
static __global__ void __launch_bounds__(256)
combine_slots(const float* __restrict__ part, float* __restrict__ out, int E, int tiles_per_head, long long total_tiles, long long P)
{
    const int e = blockIdx.x * 256 + threadIdx.x;
    if (e >= E) return;
    const int g = blockIdx.y;
    const long long c0 = tile_owner((long long)g * tiles_per_head, total_tiles, P);
    const long long c1 = tile_owner((long long)(g + 1) * tiles_per_head - 1, total_tiles, P);
    float acc = 0.f;
    for (long long cta = c0; cta <= c1; ++cta) acc += part[(size_t)(cta + g) * E + e];
    out[(size_t)g * E + e] = acc;
}

// The two steps in one for dS, dz: fixed-order sum of the (CTA, head) records, fp32 state and, for the matrix part, the
// bf16 hi and lo images the key side reads.  grid = (ceil(kE/256), G).
static __global__ void __launch_bounds__(256)
combine_slots_hilo(const float* __restrict__ part, float* __restrict__ out, __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo,
                   int tiles_per_head, long long total_tiles, long long P)
{
    const int e = blockIdx.x * 256 + threadIdx.x;
    if (e >= kE) return;
    const int g = blockIdx.y;
    const long long c0 = tile_owner((long long)g * tiles_per_head, total_tiles, P);
    const long long c1 = tile_owner((long long)(g + 1) * tiles_per_head - 1, total_tiles, P);
    float acc = 0.f;
    for (long long cta = c0; cta <= c1; ++cta) acc += part[(size_t)(cta + g) * kE + e];
    out[(size_t)g * kE + e] = acc;
    if (e < kD * kD) {
        const __nv_bfloat16 h = __float2bfloat16_rn(acc);
        hi[(size_t)g * kD * kD + e] = h;
        lo[(size_t)g * kD * kD + e] = __float2bfloat16_rn(acc - __bfloat162float(h));
    }
}

// Matrix part of a state record ([c][f] fp32) -> bf16 hi and lo images (either may be NULL).  grid = (64, G).
static __global__ void __launch_bounds__(256)
hilo_images(const float* __restrict__ state, __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo)
{
    const int e = blockIdx.x * 256 + threadIdx.x, g = blockIdx.y;
    const float x = state[(size_t)g * kE + e];
    const __nv_bfloat16 h = __float2bfloat16_rn(x);
    if (hi) hi[(size_t)g * kD * kD + e] = h;
    if (lo) lo[(size_t)g * kD * kD + e] = __float2bfloat16_rn(x - __bfloat162float(h));
}

// dW[w][c][j] = sum over the heads g that use weight matrix w (per_head: g % H == w; shared: all), ascending, and
// over the CTAs of each, ascending, of part_w[(cta + g)][j][c].  grid = (kWRec / 256, per_head ? H : 1).
static __global__ void __launch_bounds__(256)
combine_wgrad_slots(const float* __restrict__ part_w, float* __restrict__ dW, int G, int H, int per_head, int tiles_per_head,
                    long long total_tiles, long long P)
{
    const int r = blockIdx.x * 256 + threadIdx.x;   // index in a record, j * 128 + c: neighbouring threads read neighbouring words
    const int j = r / kD, cc = r % kD, wsel = blockIdx.y;
    float acc = 0.f;
    for (int g = per_head ? wsel : 0; g < G; g += per_head ? H : 1) {
        const long long c0 = tile_owner((long long)g * tiles_per_head, total_tiles, P);
        const long long c1 = tile_owner((long long)(g + 1) * tiles_per_head - 1, total_tiles, P);
        for (long long cta = c0; cta <= c1; ++cta) acc += part_w[(size_t)(cta + g) * kWRec + r];
    }
    dW[(size_t)wsel * kWRec + (size_t)cc * kM + j] = acc;
}

// Both weight gradients in one launch: blockIdx.z = 0: dW_q from part_wq, 1: dW_k from part_wk.  grid = (kWRec / 256, per_head ? H : 1, 2).
static __global__ void __launch_bounds__(256)
combine_wgrad_slots2(const float* __restrict__ part_wq, const float* __restrict__ part_wk, float* __restrict__ dWq, float* __restrict__ dWk,
                     int G, int H, int per_head, int tiles_per_head, long long total_tiles, long long P)
{
    const float* part_w = blockIdx.z == 0 ? part_wq : part_wk;
    float* dW = blockIdx.z == 0 ? dWq : dWk;
    const int r = blockIdx.x * 256 + threadIdx.x;
    const int j = r / kD, cc = r % kD, wsel = blockIdx.y;
    float acc = 0.f;
    for (int g = per_head ? wsel : 0; g < G; g += per_head ? H : 1) {
        const long long c0 = tile_owner((long long)g * tiles_per_head, total_tiles, P);
        const long long c1 = tile_owner((long long)(g + 1) * tiles_per_head - 1, total_tiles, P);
        for (long long cta = c0; cta <= c1; ++cta) acc += part_w[(size_t)(cta + g) * kWRec + r];
    }
    dW[(size_t)wsel * kWRec + (size_t)cc * kM + j] = acc;
}

}  // namespace tc
}  // namespace linattn
