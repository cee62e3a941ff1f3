// Tensor-core kernels (tcgen05 + TMEM + TMA) for linear attention with the Hedgehog feature map,
// bf16 storage, head dimension 128.  Three launches per forward:
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
// Warp roles: warps 0-3 feature map of softmax(+U) / output columns 0-63, warps 4-7 softmax(-U) / columns
// 64-127, warp 8 TMA producer, warp 9 issues the logits MMAs, warp 10 issues the accumulation MMAs, and
// (query side only) warp 11 issues the TMA stores.  Role loops are warp-uniform; single-thread work
// (TMA and MMA issue) is predicated inside them.
// Every wait is bounded: on time-out the kernel records a code in *err and unwinds.
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
constexpr int kKThreads = 352;      // key side: 11 warps
constexpr int kQThreads = 384;      // query side: 12 warps
constexpr int kE = kD * kD + kD;    // floats per (S, z) record
constexpr uint32_t kTileBytes = kTile * kD * 2;       // 32 KB: one [128 x 128] bf16 tile
constexpr uint32_t kHalfTileBytes = kTileBytes / 2;   // one 64-column block of a tile
constexpr uint32_t kWBytes = kM * kD * 2;             // 16 KB: W^T [64 x 128] bf16
constexpr uint32_t kZBlkBytes = 2 * 16 * 128;         // 4 KB: z operand, [2 blocks][16 rows][64] bf16
constexpr uint64_t kWaitLimitNs = 2000ull * 1000 * 1000;
constexpr float kLog2e = 1.4426950408889634f;

// error codes OR-ed into *err (which wait gave up)
enum : uint32_t {
    kErrProducer = 1u, kErrMmaLoad = 2u, kErrMmaU = 4u, kErrMmaPhi = 8u, kErrMmaAcc = 16u,
    kErrSoftmaxU = 32u, kErrDrain = 64u, kErrEpilogue = 128u, kErrSeg = 256u, kErrStore = 512u
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

// All lanes wait (bounded); the verdict is made warp-uniform so that role loops never diverge.
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, uint32_t* err, uint32_t code)
{
    const bool ok = mbar_wait(bar, parity, kWaitLimitNs);
    const bool all = __all_sync(0xffffffffu, ok);
    if (!all && (threadIdx.x & 31) == 0) atomicOr(err, code);
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

// One softmax half of Eq. 6 for one token.  u[64] holds the logits of this thread's token on entry.
// kNeg = false: softmax(+u); kNeg = true: softmax(-u).  The 64 results, scaled by `keep` (0 for rows
// past the end of the sequence), are written as bf16 to `row_base` = start of this token's 128-byte row
// in the 64-feature block, 16-byte chunk c stored at chunk c ^ (row & 7) (the 128-byte swizzle).
template <bool kNeg>
__device__ __forceinline__ void softmax_half_to_smem(float (&u)[kM], float keep, uint8_t* row_base, int row)
{
    float m = u[0];
#pragma unroll
    for (int j = 1; j < kM; ++j) m = kNeg ? fminf(m, u[j]) : fmaxf(m, u[j]);
    // exp(u - max) = 2^(u*log2e - max*log2e);   exp(-u - max(-u)) = 2^(min*log2e - u*log2e)
    const float mL = m * kLog2e;
    float sum = 0.f;
#pragma unroll
    for (int j = 0; j < kM; ++j) {
        const float e = kNeg ? ex2_approx(fmaf(-u[j], kLog2e, mL)) : ex2_approx(fmaf(u[j], kLog2e, -mL));
        u[j] = e;
        sum += e;
    }
    const float inv = __fdividef(keep, sum);
    const int sw = row & 7;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        uint4 v;
        v.x = pack_bf16(u[8 * c + 0] * inv, u[8 * c + 1] * inv);
        v.y = pack_bf16(u[8 * c + 2] * inv, u[8 * c + 3] * inv);
        v.z = pack_bf16(u[8 * c + 4] * inv, u[8 * c + 5] * inv);
        v.w = pack_bf16(u[8 * c + 6] * inv, u[8 * c + 7] * inv);
        *reinterpret_cast<uint4*>(row_base + ((c ^ sw) << 4)) = v;
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
#else
#define LA_TRACE(role, tile, ev) do { } while (0)
#endif

// Shared-memory descriptor with the address field replaced: descriptors of one operand family differ
// only in their start address, so the constant part is built once.
__device__ __forceinline__ uint64_t desc_at(uint64_t base_desc, uint32_t smem_addr)
{
    return base_desc | (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
}

// U = X W (Eq. 6 logits) for one tile: A = X tile (K-major), B = W^T (K-major), D = 128 x 64 fp32.
__device__ __forceinline__ void issue_logits_mma(uint32_t d_tmem, uint32_t x_smem, uint32_t w_smem)
{
    constexpr uint32_t idesc = make_idesc_bf16(kTile, kM, 0, 0);
    const uint64_t kmajor = make_desc_sw128(0, 16, 1024);
#pragma unroll
    for (int k = 0; k < kD / 16; ++k) {
        const uint64_t da = desc_at(kmajor, x_smem + (k >> 2) * kHalfTileBytes + (k & 3) * 32);
        const uint64_t db = desc_at(kmajor, w_smem + (k >> 2) * (kWBytes / 2) + (k & 3) * 32);
        mma_bf16_ss(d_tmem, da, db, idesc, k > 0);
    }
}

// ======================================================================================================
// Key side
// ======================================================================================================

constexpr int kKStages = 3;
struct KSideSmem {
    static constexpr uint32_t kStage = 2 * kTileBytes;                    // K (later phi) + V
    static constexpr uint32_t kW = kKStages * kStage;                     // 2 x W^T
    static constexpr uint32_t kOnes = kW + 2 * kWBytes;                   // 1 KB of bf16 ones
    static constexpr uint32_t kBars = kOnes + 1024;
    static constexpr uint32_t kTotal = kBars + 256 + 1024;                // + barriers + alignment slack
};

struct KSideArgs {
    float* partial;   // [slots][kE]
    uint32_t* err;
    int n, H;
    int tiles_per_head;
    long long total_tiles;
#ifdef LINATTN_TRACE
    long long* trace;
#endif
};

__global__ void __launch_bounds__(kKThreads, 1)
kside_tc(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
         const __grid_constant__ CUtensorMap tmW, const KSideArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + KSideSmem::kBars);
    enum { FULL = 0, EMPTY = 3, UFULL = 6, UEMPTY = 8, PHIFULL = 10, WFULL = 13, WFREE = 15, ACCFULL = 17, ACCFREE = 18, NBARS = 19 };
    const uint32_t bar0 = smem_u32(bars);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(&bars[NBARS]);
    uint32_t* err = a.err;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int i = 0; i < kKStages; ++i) { mbar_init(bar(FULL + i), 1); mbar_init(bar(EMPTY + i), 1); mbar_init(bar(PHIFULL + i), 8); }
        for (int i = 0; i < 2; ++i) { mbar_init(bar(UFULL + i), 1); mbar_init(bar(UEMPTY + i), 8); mbar_init(bar(WFULL + i), 1); mbar_init(bar(WFREE + i), 1); }
        mbar_init(bar(ACCFULL), 1);
        mbar_init(bar(ACCFREE), 8);
        fence_mbar_init();
    }
    if (warp == 9) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    if (warp == 8 && lane == 0) {
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
        tma_prefetch_desc(&tmW);
    }
    for (int i = tid; i < 512; i += kKThreads) reinterpret_cast<__nv_bfloat16*>(smem + KSideSmem::kOnes)[i] = __float2bfloat16(1.0f);
    fence_proxy_async_smem();
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t tmem_u = tmem;            // 2 x 64 columns of logits
    const uint32_t tmem_s = tmem + 128;      // 128 columns: S[f][c], lane = f
    const uint32_t tmem_z = tmem + 256;      // 16 columns: z[f] (all 16 equal)

    TileWalk w;
    w.init(a.total_tiles, a.tiles_per_head);

    if (warp == 8) {
        // ---------------- TMA producer ----------------
        Ring<kKStages> r;
        int issued = 0;
        for (; !w.done(); w.next(), r.next()) {
            if (w.first()) {
                const int wb = w.seg & 1;
                if (w.seg >= 2 && !warp_wait(bar(WFREE + wb), ((w.seg >> 1) - 1) & 1, err, kErrProducer)) break;
                if (lane == 0) {
                    mbar_arrive_expect_tx(bar(WFULL + wb), kWBytes);
                    const uint32_t wdst = sbase + KSideSmem::kW + wb * kWBytes;
                    tma_load_3d(wdst, &tmW, bar(WFULL + wb), 0, 0, w.g % a.H);
                    tma_load_3d(wdst + kWBytes / 2, &tmW, bar(WFULL + wb), 64, 0, w.g % a.H);
                }
            }
            if (w.i >= kKStages && !warp_wait(bar(EMPTY + r.s), r.ph ^ 1u, err, kErrProducer)) break;
            LA_TRACE(0, w.i, 0);
            if (lane == 0) {
                mbar_arrive_expect_tx(bar(FULL + r.s), 2 * kTileBytes);
                const uint32_t kdst = sbase + r.s * KSideSmem::kStage, vdst = kdst + kTileBytes;
                tma_load_3d(kdst, &tmK, bar(FULL + r.s), 0, w.lt * kTile, w.g);
                tma_load_3d(kdst + kHalfTileBytes, &tmK, bar(FULL + r.s), 64, w.lt * kTile, w.g);
                tma_load_3d(vdst, &tmV, bar(FULL + r.s), 0, w.lt * kTile, w.g);
                tma_load_3d(vdst + kHalfTileBytes, &tmV, bar(FULL + r.s), 64, w.lt * kTile, w.g);
            }
            issued = w.i + 1;
        }
        if (issued < w.count) {
            // unwinding after a time-out: let the copies already in flight land before the CTA exits
            for (int i = (issued > kKStages ? issued - kKStages : 0); i < issued; ++i)
                mbar_wait(bar(FULL + i % kKStages), (uint32_t)(i / kKStages) & 1u, kWaitLimitNs);
        }
    } else if (warp == 9) {
        // ---------------- logits MMA issuer: U = K W_k ----------------
        Ring<kKStages> r;
        Ring<2> ur;
        for (; !w.done(); w.next(), r.next(), ur.next()) {
            const int wb = w.seg & 1;
            if (w.first() && !warp_wait(bar(WFULL + wb), (uint32_t)(w.seg >> 1) & 1u, err, kErrMmaLoad)) break;
            if (!warp_wait(bar(FULL + r.s), r.ph, err, kErrMmaLoad)) break;
            LA_TRACE(1, w.i, 0);
            if (w.i >= 2 && !warp_wait(bar(UEMPTY + ur.s), ur.ph ^ 1u, err, kErrMmaU)) break;
            tcgen05_fence_after();
            if (elect_one()) {
                issue_logits_mma(tmem_u + ur.s * kM, sbase + r.s * KSideSmem::kStage, sbase + KSideSmem::kW + wb * kWBytes);
                mma_commit(bar(UFULL + ur.s));
                if (w.last()) mma_commit(bar(WFREE + wb));
            }
            __syncwarp();
            LA_TRACE(1, w.i, 1);
        }
    } else if (warp == 10) {
        // ---------------- accumulation MMA issuer: S += phi^T V, z += phi^T 1 ----------------
        constexpr uint32_t idesc_s = make_idesc_bf16(kD, kD, 1, 1);   // A = phi^T (MN-major), B = V (MN-major)
        constexpr uint32_t idesc_z = make_idesc_bf16(kD, 16, 1, 0);   // B = ones (K-major, no swizzle)
        const uint64_t ones_desc = make_desc_noswizzle(sbase + KSideSmem::kOnes, 128, 256);
        const uint64_t mnmajor = make_desc_sw128(0, kHalfTileBytes, 1024);
        Ring<kKStages> r;
        for (; !w.done(); w.next(), r.next()) {
            if (!warp_wait(bar(PHIFULL + r.s), r.ph, err, kErrMmaPhi)) break;
            LA_TRACE(1, w.i, 2);
            const bool first = w.first();
            if (first && w.seg >= 1 && !warp_wait(bar(ACCFREE), (uint32_t)(w.seg - 1) & 1u, err, kErrMmaAcc)) break;
            tcgen05_fence_after();
            if (elect_one()) {
                const uint32_t phi = sbase + r.s * KSideSmem::kStage, vt = phi + kTileBytes;
#pragma unroll
                for (int k = 0; k < kTile / 16; ++k) {
                    const uint64_t da = desc_at(mnmajor, phi + k * 2048);
                    const uint64_t db = desc_at(mnmajor, vt + k * 2048);
                    const uint32_t acc = (first && k == 0) ? 0u : 1u;
                    mma_bf16_ss(tmem_s, da, db, idesc_s, acc);
                    mma_bf16_ss(tmem_z, da, ones_desc, idesc_z, acc);
                }
                mma_commit(bar(EMPTY + r.s));
                if (w.last()) mma_commit(bar(ACCFULL));
            }
            __syncwarp();
            LA_TRACE(1, w.i, 3);
        }
    } else {
        // ---------------- feature map + drain (warps 0-7) ----------------
        const int half = warp >> 2;                       // 0: softmax(+U), 1: softmax(-U)
        const int row = (warp & 3) * 32 + lane;           // token within the tile == TMEM lane
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        Ring<kKStages> r;
        Ring<2> ur;
        for (; !w.done(); w.next(), r.next(), ur.next()) {
            if (!warp_wait(bar(UFULL + ur.s), ur.ph, err, kErrSoftmaxU)) break;
            if ((warp & 3) == 0) LA_TRACE(2 + half, w.i, 0);
            tcgen05_fence_after();
            float u[kM];
            load_logits(tmem_u + lane_base + ur.s * kM, u);
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(UEMPTY + ur.s));
            if ((warp & 3) == 0) LA_TRACE(2 + half, w.i, 1);
            const float keep = (w.lt * kTile + row < a.n) ? 1.f : 0.f;
            uint8_t* dst = smem + r.s * KSideSmem::kStage + half * kHalfTileBytes + row * 128;
            if (half == 0) softmax_half_to_smem<false>(u, keep, dst, row);
            else softmax_half_to_smem<true>(u, keep, dst, row);
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(PHIFULL + r.s));
            if ((warp & 3) == 0) LA_TRACE(2 + half, w.i, 2);
            if (w.last()) {
                // drain the accumulators of this segment: thread = feature f, this half's 64 columns of S
                if (!warp_wait(bar(ACCFULL), (uint32_t)w.seg & 1u, err, kErrDrain)) break;
                tcgen05_fence_after();
                float* rec = a.partial + (size_t)(blockIdx.x + w.g) * kE;
                float* srow = rec + (size_t)row * kD + half * 64;
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld_x32(tmem_s + lane_base + half * 64 + c0, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int q4 = 0; q4 < 8; ++q4)
                        *reinterpret_cast<uint4*>(srow + c0 + 4 * q4) = make_uint4(v[4 * q4], v[4 * q4 + 1], v[4 * q4 + 2], v[4 * q4 + 3]);
                }
                if (half == 0) {
                    uint32_t zr[2];
                    tmem_ld_x2(tmem_z + lane_base, zr);
                    tmem_wait_ld();
                    rec[kD * kD + row] = __uint_as_float(zr[0]);
                }
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(ACCFREE));
            }
        }
    }
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 9) tmem_dealloc(tmem, 512);
}

// ======================================================================================================
// Combine
// ======================================================================================================

struct CombineArgs {
    const float* partial;       // [slots][kE]
    float* state;               // [G][kE] fp32 (S row-major [f][c], then z)
    __nv_bfloat16* s_img;       // [G][128][128] bf16, S[f][c] row-major
    __nv_bfloat16* z_img;       // [G][2][16][64] bf16 operand image: row 0 = hi(z), row 1 = lo(z), swizzled
    long long tiles_per_head, total_tiles, P;
};

// grid = (ceil(kE / 256), G).  Sums the partials of head g over the CTAs that touched it, in CTA order.
static __global__ void __launch_bounds__(256) combine_tc(const CombineArgs a)
{
    const int e = blockIdx.x * 256 + threadIdx.x;
    if (e >= kE) return;
    const long long g = blockIdx.y;
    const long long c0 = tile_owner(g * a.tiles_per_head, a.total_tiles, a.P);
    const long long c1 = tile_owner((g + 1) * a.tiles_per_head - 1, a.total_tiles, a.P);
    const float* p = a.partial + (size_t)(c0 + g) * kE + e;
    const int cnt = (int)(c1 - c0) + 1;
    float acc = 0.f;
    int c = 0;
    for (; c + 8 <= cnt; c += 8) {  // loads first (independent), then the adds in CTA order
        float v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = p[(size_t)(c + u) * kE];
#pragma unroll
        for (int u = 0; u < 8; ++u) acc += v[u];
    }
    for (; c < cnt; ++c) acc += p[(size_t)c * kE];
    a.state[(size_t)g * kE + e] = acc;
    if (e < kD * kD) {
        a.s_img[(size_t)g * kD * kD + e] = __float2bfloat16_rn(acc);
    } else {
        // z[f]: hi and lo bf16 parts into rows 0 and 1 of the K-major operand block of feature block f / 64
        const int f = e - kD * kD;
        const __nv_bfloat16 hi = __float2bfloat16_rn(acc);
        const __nv_bfloat16 lo = __float2bfloat16_rn(acc - __bfloat162float(hi));
        __nv_bfloat16* blk = a.z_img + (size_t)g * (kZBlkBytes / 2) + (f >> 6) * (16 * 64);
        const int fi = f & 63, chunk = fi >> 3, within = fi & 7;
        blk[0 * 64 + ((chunk ^ 0) << 3) + within] = hi;  // row 0: swizzle term (row & 7) = 0
        blk[1 * 64 + ((chunk ^ 1) << 3) + within] = lo;  // row 1: swizzle term 1
    }
}

// ======================================================================================================
// Query side
// ======================================================================================================

constexpr int kQStages = 5;
struct QSideSmem {
    static constexpr uint32_t kS = kQStages * kTileBytes;   // S image (32 KB)
    static constexpr uint32_t kW = kS + kTileBytes;         // W^T (16 KB)
    static constexpr uint32_t kZ = kW + kWBytes;            // z operand (4 KB)
    static constexpr uint32_t kBars = kZ + kZBlkBytes;
    static constexpr uint32_t kTotal = kBars + 512 + 1024;
};

struct QSideArgs {
    const __nv_bfloat16* z_img;  // [G][kZBlkBytes / 2]
    uint32_t* err;
    int n, H;
    int tiles_per_head;
    long long total_tiles;
#ifdef LINATTN_TRACE
    long long* trace;
#endif
};

__device__ __forceinline__ void bulk_load_1d(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

__global__ void __launch_bounds__(kQThreads, 1)
qside_tc(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmO,
         const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmS, const QSideArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + QSideSmem::kBars);
    enum { QFULL = 0, QEMPTY = 5, PHIFULL = 10, OFULL = 15, UFULL = 20, UEMPTY = 22, DFULL = 24, DEMPTY = 26, SEGFULL = 28, SEGFREE = 29, NBARS = 30 };
    const uint32_t bar0 = smem_u32(bars);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(&bars[NBARS]);
    uint32_t* err = a.err;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int i = 0; i < kQStages; ++i) { mbar_init(bar(QFULL + i), 1); mbar_init(bar(QEMPTY + i), 1); mbar_init(bar(PHIFULL + i), 8); mbar_init(bar(OFULL + i), 8); }
        for (int i = 0; i < 2; ++i) { mbar_init(bar(UFULL + i), 1); mbar_init(bar(UEMPTY + i), 8); mbar_init(bar(DFULL + i), 1); mbar_init(bar(DEMPTY + i), 8); }
        mbar_init(bar(SEGFULL), 1);
        mbar_init(bar(SEGFREE), 1);
        fence_mbar_init();
    }
    if (warp == 9) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    if (warp == 8 && lane == 0) {
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmO);
        tma_prefetch_desc(&tmW);
        tma_prefetch_desc(&tmS);
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t tmem_u = tmem;  // 2 x 64 columns of logits
    auto tmem_num = [&](int db) { return tmem + 128 + db * 160; };   // 128 columns: num[token][c]
    auto tmem_den = [&](int db) { return tmem + 256 + db * 160; };   // 16 columns: [hi(z) part, lo(z) part, ...]

    TileWalk w;
    w.init(a.total_tiles, a.tiles_per_head);

    if (warp == 8) {
        // ---------------- TMA producer ----------------
        Ring<kQStages> r;
        int issued = 0;
        for (; !w.done(); w.next(), r.next()) {
            if (w.first()) {
                if (w.seg >= 1 && !warp_wait(bar(SEGFREE), (uint32_t)(w.seg - 1) & 1u, err, kErrSeg)) break;
                if (lane == 0) {
                    mbar_arrive_expect_tx(bar(SEGFULL), kWBytes + kTileBytes + kZBlkBytes);
                    tma_load_3d(sbase + QSideSmem::kW, &tmW, bar(SEGFULL), 0, 0, w.g % a.H);
                    tma_load_3d(sbase + QSideSmem::kW + kWBytes / 2, &tmW, bar(SEGFULL), 64, 0, w.g % a.H);
                    tma_load_3d(sbase + QSideSmem::kS, &tmS, bar(SEGFULL), 0, 0, w.g);
                    tma_load_3d(sbase + QSideSmem::kS + kHalfTileBytes, &tmS, bar(SEGFULL), 64, 0, w.g);
                    bulk_load_1d(sbase + QSideSmem::kZ, a.z_img + (size_t)w.g * (kZBlkBytes / 2), kZBlkBytes, bar(SEGFULL));
                }
            }
            if (w.i >= kQStages && !warp_wait(bar(QEMPTY + r.s), r.ph ^ 1u, err, kErrProducer)) break;
            if (lane == 0) {
                mbar_arrive_expect_tx(bar(QFULL + r.s), kTileBytes);
                tma_load_3d(sbase + r.s * kTileBytes, &tmQ, bar(QFULL + r.s), 0, w.lt * kTile, w.g);
                tma_load_3d(sbase + r.s * kTileBytes + kHalfTileBytes, &tmQ, bar(QFULL + r.s), 64, w.lt * kTile, w.g);
            }
            issued = w.i + 1;
        }
        if (issued < w.count) {
            for (int i = (issued > kQStages ? issued - kQStages : 0); i < issued; ++i)
                mbar_wait(bar(QFULL + i % kQStages), (uint32_t)(i / kQStages) & 1u, kWaitLimitNs);
        }
    } else if (warp == 9) {
        // ---------------- logits MMA issuer: U = Q W_q ----------------
        Ring<kQStages> r;
        Ring<2> ur;
        for (; !w.done(); w.next(), r.next(), ur.next()) {
            if (w.first() && !warp_wait(bar(SEGFULL), (uint32_t)w.seg & 1u, err, kErrSeg)) break;
            if (!warp_wait(bar(QFULL + r.s), r.ph, err, kErrMmaLoad)) break;
            if (w.i >= 2 && !warp_wait(bar(UEMPTY + ur.s), ur.ph ^ 1u, err, kErrMmaU)) break;
            tcgen05_fence_after();
            if (elect_one()) {
                issue_logits_mma(tmem_u + ur.s * kM, sbase + r.s * kTileBytes, sbase + QSideSmem::kW);
                mma_commit(bar(UFULL + ur.s));
            }
            __syncwarp();
        }
    } else if (warp == 10) {
        // ---------------- numerator / denominator MMA issuer: num = phi(q) S, den = phi(q) . z ----------------
        constexpr uint32_t idesc_n = make_idesc_bf16(kTile, kD, 0, 1);   // A = phi(q) (K-major), B = S (MN-major)
        constexpr uint32_t idesc_d = make_idesc_bf16(kTile, 16, 0, 0);   // B = z operand (K-major)
        const uint64_t kmajor = make_desc_sw128(0, 16, 1024);
        const uint64_t mnmajor = make_desc_sw128(0, kHalfTileBytes, 1024);
        Ring<kQStages> r;
        Ring<2> dr;
        for (; !w.done(); w.next(), r.next(), dr.next()) {
            if (w.first() && !warp_wait(bar(SEGFULL), (uint32_t)w.seg & 1u, err, kErrSeg)) break;
            if (!warp_wait(bar(PHIFULL + r.s), r.ph, err, kErrMmaPhi)) break;
            if (w.i >= 2 && !warp_wait(bar(DEMPTY + dr.s), dr.ph ^ 1u, err, kErrMmaAcc)) break;
            tcgen05_fence_after();
            if (elect_one()) {
                const uint32_t phi = sbase + r.s * kTileBytes;
#pragma unroll
                for (int k = 0; k < kD / 16; ++k) {
                    const uint64_t da = desc_at(kmajor, phi + (k >> 2) * kHalfTileBytes + (k & 3) * 32);
                    const uint64_t db_s = desc_at(mnmajor, sbase + QSideSmem::kS + k * 2048);
                    const uint64_t db_z = desc_at(kmajor, sbase + QSideSmem::kZ + (k >> 2) * 2048 + (k & 3) * 32);
                    mma_bf16_ss(tmem_num(dr.s), da, db_s, idesc_n, k > 0);
                    mma_bf16_ss(tmem_den(dr.s), da, db_z, idesc_d, k > 0);
                }
                mma_commit(bar(DFULL + dr.s));
                if (w.last()) mma_commit(bar(SEGFREE));   // this head's S, z and W may now be replaced
            }
            __syncwarp();
        }
    } else if (warp == 11) {
        // ---------------- TMA stores of finished output tiles ----------------
        Ring<kQStages> r;
        for (; !w.done(); w.next(), r.next()) {
            if (!warp_wait(bar(OFULL + r.s), r.ph, err, kErrStore)) break;
            if (lane == 0) {
                tma_store_3d(&tmO, sbase + r.s * kTileBytes, 0, w.lt * kTile, w.g);
                tma_store_3d(&tmO, sbase + r.s * kTileBytes + kHalfTileBytes, 64, w.lt * kTile, w.g);
                bulk_commit_group();
                bulk_wait_group_read<0>();   // the slot has been read out: hand it back to the producer
                mbar_arrive(bar(QEMPTY + r.s));
            }
            __syncwarp();
        }
        if (lane == 0) bulk_wait_group<0>();
    } else {
        // ---------------- feature map + epilogue (warps 0-7) ----------------
        const int half = warp >> 2;
        const int row = (warp & 3) * 32 + lane;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        Ring<kQStages> r, er;   // feature-map ring position, epilogue ring position (one tile behind)
        Ring<2> ur, dr;
        for (int i = 0; i <= w.count; ++i) {
            if (i < w.count) {
                if (!warp_wait(bar(UFULL + ur.s), ur.ph, err, kErrSoftmaxU)) break;
                tcgen05_fence_after();
                float u[kM];
                load_logits(tmem_u + lane_base + ur.s * kM, u);
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(UEMPTY + ur.s));
                uint8_t* dst = smem + r.s * kTileBytes + half * kHalfTileBytes + row * 128;
                if (half == 0) softmax_half_to_smem<false>(u, 1.f, dst, row);
                else softmax_half_to_smem<true>(u, 1.f, dst, row);
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(PHIFULL + r.s));
                r.next();
                ur.next();
            }
            if (i >= 1) {
                if (!warp_wait(bar(DFULL + dr.s), dr.ph, err, kErrEpilogue)) break;
                tcgen05_fence_after();
                uint32_t v[64], dv[2];
                tmem_ld_x32(tmem_num(dr.s) + lane_base + half * 64, v);
                tmem_ld_x32(tmem_num(dr.s) + lane_base + half * 64 + 32, v + 32);
                tmem_ld_x2(tmem_den(dr.s) + lane_base, dv);
                tmem_wait_ld();
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(DEMPTY + dr.s));
                const float inv = __fdividef(1.f, __uint_as_float(dv[0]) + __uint_as_float(dv[1]));
                uint8_t* dst = smem + er.s * kTileBytes + half * kHalfTileBytes + row * 128;
                const int sw = row & 7;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    uint4 o;
                    o.x = pack_bf16(__uint_as_float(v[8 * c + 0]) * inv, __uint_as_float(v[8 * c + 1]) * inv);
                    o.y = pack_bf16(__uint_as_float(v[8 * c + 2]) * inv, __uint_as_float(v[8 * c + 3]) * inv);
                    o.z = pack_bf16(__uint_as_float(v[8 * c + 4]) * inv, __uint_as_float(v[8 * c + 5]) * inv);
                    o.w = pack_bf16(__uint_as_float(v[8 * c + 6]) * inv, __uint_as_float(v[8 * c + 7]) * inv);
                    *reinterpret_cast<uint4*>(dst + ((c ^ sw) << 4)) = o;
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(OFULL + er.s));
                er.next();
                dr.next();
            }
        }
    }
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 9) tmem_dealloc(tmem, 512);
}

// W [H][128 d][64 j] (any supported type) -> W^T bf16 [H][64 j][128 d]; per_head == 0 replicates one matrix.
template <typename T>
static __global__ void transpose_weights_bf16(const T* __restrict__ src, __nv_bfloat16* __restrict__ dst, int H, int per_head)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)H * kM * kD) return;
    const int h = (int)(i / (kM * kD)), rem = (int)(i % (kM * kD)), j = rem / kD, dd = rem % kD;
    const size_t s = (size_t)(per_head ? h : 0) * kD * kM + (size_t)dd * kM + j;
    dst[i] = __float2bfloat16_rn((float)src[s]);
}

}  // namespace tc
}  // namespace linattn
