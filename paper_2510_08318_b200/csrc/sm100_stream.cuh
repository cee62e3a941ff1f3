// The whole forward of linear attention with the Hedgehog feature map (Eq. 5, Eq. 6) as ONE persistent
// cooperative kernel, bf16 storage, head dimension 128.  Each CTA walks one list of 128-token work items,
//
//     key items of wave 0, key items of wave 1, query items of wave 0, query items of wave 1
//
// (a wave is a contiguous range of (batch, head) pairs; there are one or two), and every item flows through the
// same pipeline of warp roles with no CTA-wide drain between the key side and the query side:
//
//   warp 8      TMA producer: K and V tiles (key item) or a Q tile (query item) into a ring of six 32 KB
//               slots; W_k / W_q per head; the bf16 image of S and fp32 z per head for query items
//   warp 9      logits U = X W (tcgen05.mma, 128 x 64 x 128, fp32 in TMEM)                               Eq. 6
//   warps 0-7   phi = softmax(U) (+) softmax(-U), one token per thread, bf16, written over the X tile;
//               for query items also the denominator phi(q) . z (fp32), handed over through TMEM        Eq. 6, Eq. 5
//   warp 10     key item:   S += phi(k)^T V into a TMEM accumulator that lives for the whole (CTA, head) run
//               query item: num = phi(q) S                                                              Eq. 5
//   warps 12-15 key item:   z += column sums of phi(k) (CUDA cores); at the end of a run, the accumulator and z
//                           go to this CTA's partial record of the head
//               query item: o = num / den -> bf16 over the tile in its slot                               Eq. 5
//               in between: their share of the fixed-order sum of a wave's partial records into S and z
//   warp 11     TMA stores of finished output tiles
//
// Dependencies between CTAs are two monotonic counters per wave in global memory: "key side done" (every
// CTA has written its partial records of the wave) and "combined" (S and z of the wave's heads are final).
// With two waves the query items of wave 0 start right behind the key items of wave 1, long after wave 0
// was combined, and wave 1 is combined while the query items of wave 0 stream: no CTA ever idles at a
// grid-wide barrier.  All CTAs must be co-resident (cooperative launch).  Every wait is bounded.
#pragma once
#include "sm100_kernels.cuh"

namespace linattn {
namespace tc {

constexpr int kSlots = 6;                        // 32 KB slots; a key item takes two (K, V), a query item one
constexpr int kQRing = 5;                        // query items cycle through slots 0..4; slot 5 holds the S image
constexpr int kSSlot = 5;
constexpr int kRec = kD * kD + 4 * kD;           // floats per partial record: S, then z as four token-quarter parts
constexpr int kQuadsPerHead = kD * kD / 4 + kD / 4;  // combine work items per head: float4 groups of S, of z
constexpr uint32_t kTmemU = 0, kTmemAcc = 128, kTmemDen = 384;   // TMEM columns: 2x64 logits, 2x128 accumulators, 16 denominators

struct SmemStream {
    static constexpr uint32_t kW = kSlots * kTileBytes;     // 2 x W^T (16 KB each), by run parity
    static constexpr uint32_t kZ = kW + 2 * kWBytes;        // z of the current query run, fp32 [128]
    static constexpr uint32_t kBars = kZ + 512;             // mbarriers, TMEM slot, abort word
    static constexpr uint32_t kTotal = kBars + 512 + 1024;  // + alignment slack
};

// mbarrier indices
enum : int {
    S_FULL = 0,      // [6] TMA loads of the item in this slot have landed (key item: K and V, on the K slot)
    S_EMPTY = 6,     // [6] the tensor core / the TMA store is done reading the slot
    S_PHI = 12,      // [6] phi has been written over the X tile (8 feature-map warps)
    S_OUT = 18,      // [6] the output tile is in the slot (4 epilogue warps)
    S_AUX = 24,      // [3] key item in slots (2i, 2i+1): the z column sums have read phi (4 warps)
    S_UFULL = 27, S_UEMPTY = 29,     // [2] logits buffers in TMEM
    S_WFULL = 31, S_WFREE = 33,      // [2] W^T buffers
    S_ACCFULL = 35, S_ACCFREE = 37,  // [2] TMEM accumulators
    S_STATE = 39,    // S image and z of the current query run have landed
    S_STATEFREE = 40,  // ... and are no longer needed
    S_NBARS = 41
};

struct StreamArgs {
    float* partial;        // [records][kRec]
    float* state;          // [G][kE] fp32 S as [c][f] (c = column of V, f = feature), then z
    __nv_bfloat16* s_img;  // [G][128][128] bf16 image of S, [c][f]
    uint32_t* err;         // error word
    uint32_t* cnt;         // [0..1] key-side-done counters per wave, [2..3] combined counters per wave (monotonic)
    uint32_t kdone_target[2], cdone_target[2];  // values the counters reach when this launch's wave is done
    int n, H, G, tph;      // tph = tiles per head
    int waves, gsplit;     // wave 0 = heads [0, gsplit), wave 1 = [gsplit, G); gsplit == G when waves == 1
#ifdef LINATTN_TRACE
    long long* trace;
#endif
};

// 64-bit divisions, kept out of line: they run a handful of times per role and would otherwise be
// inlined at every use.
__device__ __noinline__ longlong2 cta_range(long long T, unsigned P, unsigned c)   // CTA c's share [x, y) of T tiles
{
    return make_longlong2((long long)c * T / P, (long long)(c + 1) * T / P);
}
__device__ __noinline__ int2 split_tile(long long t, int tph)   // (head, tile within the head) of wave-local tile t
{
    return make_int2((int)(t / tph), (int)(t % tph));
}

// Heads, tiles and partial records of a wave.
struct WaveGeom {
    int g0, heads;
    long long T;        // tiles in the wave
    int rec_base;       // first partial record of the wave
    __device__ __forceinline__ void init(const StreamArgs& s, int w)
    {
        g0 = w == 0 ? 0 : s.gsplit;
        heads = (w == 0 ? s.gsplit : s.G) - g0;
        T = (long long)heads * s.tph;
        rec_base = w == 0 ? 0 : (int)gridDim.x + s.gsplit;
    }
};

// Walks this CTA's items in pipeline order.  Every role runs the same walk, so slot numbers, buffer
// parities and run boundaries agree between roles without any communication.
struct ItemWalk {
    int phase, nphase, waves;   // phase < waves: key items of wave `phase`; else query items of wave `phase - waves`
    long long t, e;             // wave-local tile index, end of this CTA's range
    int tph, g0;
    int g, lt;                  // (batch, head) index and tile within the head
    int i, ki, qi;              // items, key items, query items before this one
    int run, krun;              // runs = maximal stretches of one kind within one head ((CTA, head) pieces)
    int rp;                     // ring position
    bool is_q, run_first;
    const StreamArgs* s;

    __device__ __forceinline__ void load_phase()
    {
        for (; phase < nphase; ++phase) {
            WaveGeom wg;
            wg.init(*s, phase % waves);
            const longlong2 r = cta_range(wg.T, gridDim.x, blockIdx.x);
            if (r.y > r.x) {
                t = r.x;
                e = r.y;
                g0 = wg.g0;
                is_q = phase >= waves;
                const int2 gl = split_tile(t, tph);
                g = g0 + gl.x;
                lt = gl.y;
                run_first = true;
                return;
            }
        }
    }
    __device__ __forceinline__ void init(const StreamArgs& sa)
    {
        s = &sa;
        waves = sa.waves;
        nphase = 2 * sa.waves;
        tph = sa.tph;
        phase = 0;
        i = ki = qi = 0;
        run = krun = 0;
        rp = 0;
        is_q = false;
        load_phase();
    }
    __device__ __forceinline__ bool done() const { return phase >= nphase; }
    __device__ __forceinline__ int wave() const { return phase % waves; }
    __device__ __forceinline__ bool first() const { return run_first; }                        // first item of its run
    __device__ __forceinline__ bool last() const { return t == e - 1 || lt == tph - 1; }       // last item of its run
    __device__ __forceinline__ bool last_key_of_wave() const { return !is_q && t == e - 1; }
    __device__ __forceinline__ int slot() const { return rp; }                                 // X tile (K or Q); V is slot() + 1
    __device__ __forceinline__ int acc() const { return is_q ? (qi & 1) : (krun & 1); }        // TMEM accumulator of this item
    __device__ __forceinline__ void next()
    {
        const bool was_last = last();
        ++i;
        if (is_q) {
            ++qi;
            rp = rp + 1 == kQRing ? 0 : rp + 1;
        } else {
            ++ki;
            rp = rp + 2 == kSlots ? 0 : rp + 2;
        }
        if (was_last) {
            ++run;
            if (!is_q) ++krun;
        }
        run_first = was_last;
        ++t;
        if (t == e) {
            ++phase;
            load_phase();
            return;
        }
        if (++lt == tph) {
            lt = 0;
            ++g;
        }
    }
};

__device__ __forceinline__ void tmem_st_x1(uint32_t taddr, uint32_t v)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x1.b32 [%0], {%1};" ::"r"(taddr), "r"(v) : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ bool counter_reached(const uint32_t* p, uint32_t target)
{
    return (int32_t)(ld_acquire_gpu(p) - target) >= 0;
}

// Per-role barrier bookkeeping: one parity bit per mbarrier, flipped after every completed wait.
struct Parity {
    uint64_t bits = 0;
    __device__ __forceinline__ uint32_t get(int b) const { return (uint32_t)(bits >> b) & 1u; }
    __device__ __forceinline__ void flip(int b) { bits ^= 1ull << b; }
};

// One softmax half of Eq. 6 for one token, in a single copy of the code for all four cases (instruction
// cache footprint matters more here than the few predicated instructions):
//   neg    : false -> softmax(+u), true -> softmax(-u)
//   keep   : 1, or 0 for key rows past the end of the sequence (phi = 0 adds nothing to S and z)
//   z_half : query items only (else nullptr): this half's 64 entries of z in shared memory; the return value
//            is then this half's part of the denominator of Eq. 5, sum_f phi[f] z[f] (fp32).
// The 64 results go to `row_base` as bf16, 16-byte chunk c at chunk c ^ (row & 7) (the 128-byte swizzle).
// Arithmetic is fp32, two lanes per instruction; one pair in four takes its exponentials on the FMA pipe.
__device__ __forceinline__ float softmax_half(float (&u)[kM], bool neg, float keep, const float* z_half, uint8_t* row_base, int row)
{
    float m;
    if (neg) {
        m = min3(u[0], u[1], u[2]);
#pragma unroll
        for (int j = 3; j < kM - 1; j += 2) m = min3(m, u[j], u[j + 1]);
        m = fminf(m, u[kM - 1]);
    } else {
        m = max3(u[0], u[1], u[2]);
#pragma unroll
        for (int j = 3; j < kM - 1; j += 2) m = max3(m, u[j], u[j + 1]);
        m = fmaxf(m, u[kM - 1]);
    }
    // exp(u - max u) = 2^(u*L - max*L);   exp(-u - max(-u)) = 2^(u*(-L) - min*(-L)),  L = log2(e)
    const float sL = neg ? -kLog2e : kLog2e;
    const float off = -m * sL;
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
    const float inv1 = __fdividef(1.f, s0 + s1);
    float den = 0.f;
    if (z_half != nullptr) {
        f32x2 dot2 = pack2(0.f, 0.f);
        const ulonglong2* z4 = reinterpret_cast<const ulonglong2*>(z_half);
#pragma unroll
        for (int p = 0; p < kM / 2; p += 2) {
            const ulonglong2 zz = z4[p >> 1];   // z[2p .. 2p+3], the same address in every lane (broadcast)
            dot2 = fma2(e[p], zz.x, dot2);
            dot2 = fma2(e[p + 1], zz.y, dot2);
        }
        float d0, d1;
        unpack2(dot2, d0, d1);
        den = (d0 + d1) * inv1;
    }
    const float inv = inv1 * keep;
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
    return den;
}

// ---- combine: fixed-order sum of a wave's partial records ---------------------------------------------

// Work item x of wave `w`: one float4 group of S or of z of one head, summed over the partial records of the
// CTAs that touched the head.  Two neighbouring lanes share an item: lane `half` = 0 sums the first half of
// the records, lane 1 the second half, each in ascending CTA order (and, for z, token quarter 0..3 inside a
// record), and the result is (first half) + (second half): a fixed order, so the bits do not depend on timing.
// All loads of a lane are in flight together (one round trip to L2 for up to 16 of them).
// Must be called by all 32 lanes; lanes without an item pass valid = false.
__device__ __noinline__ void combine_item(const StreamArgs& s, int w, int x, int half, bool valid)
{
    constexpr int kBatch = 16;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    int g = 0, r = 0;
    if (valid) {
        WaveGeom wg;
        wg.init(s, w);
        const long long P = gridDim.x;
        const int gl = x / kQuadsPerHead;
        r = x % kQuadsPerHead;
        g = wg.g0 + gl;
        const long long c0 = tile_owner((long long)gl * s.tph, wg.T, P);
        const long long c1 = tile_owner((long long)(gl + 1) * s.tph - 1, wg.T, P);
        const int cnt = (int)(c1 - c0) + 1, h = (cnt + 1) >> 1;
        const int j0 = half == 0 ? 0 : h, j1 = half == 0 ? h : cnt;
        const float* rec = s.partial + (size_t)(wg.rec_base + c0 + gl) * kRec;
        const bool is_s = r < kD * kD / 4;
        const int sh = is_s ? 0 : 2;   // a z item reads four token-quarter parts per record
        const float4* p = reinterpret_cast<const float4*>(is_s ? rec + r * 4 : rec + kD * kD + (r - kD * kD / 4) * 4);
        const int nload = (j1 - j0) << sh;
        for (int base = 0; base < nload; base += kBatch) {
            float4 v[kBatch];
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const int q = base + u;
                v[u] = q < nload ? __ldcg(p + (size_t)(j0 + (q >> sh)) * (kRec / 4) + (q & ((1 << sh) - 1)) * (kD / 4))
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                if (base + u < nload) {
                    acc.x += v[u].x;
                    acc.y += v[u].y;
                    acc.z += v[u].z;
                    acc.w += v[u].w;
                }
            }
        }
    }
    float4 hi;
    hi.x = __shfl_down_sync(0xffffffffu, acc.x, 1);
    hi.y = __shfl_down_sync(0xffffffffu, acc.y, 1);
    hi.z = __shfl_down_sync(0xffffffffu, acc.z, 1);
    hi.w = __shfl_down_sync(0xffffffffu, acc.w, 1);
    if (valid && half == 0) {
        acc.x += hi.x;
        acc.y += hi.y;
        acc.z += hi.z;
        acc.w += hi.w;
        // flat index in the record == flat index in the state: S as [c][f] (c = column of V, f = feature), then z
        const int e4 = r * 4;
        *reinterpret_cast<float4*>(s.state + (size_t)g * kE + e4) = acc;
        if (r < kD * kD / 4) {
            uint2 packed;
            packed.x = pack_bf16(acc.x, acc.y);
            packed.y = pack_bf16(acc.z, acc.w);
            *reinterpret_cast<uint2*>(s.s_img + (size_t)g * kD * kD + e4) = packed;
        }
    }
}

// State of the combine duty of one aux warp: which wave is next and how far this warp's share has got.
struct CombineDuty {
    int wave = 0, step = 0;
    int published = 0;        // waves whose key side this CTA has published; a later wave cannot be complete yet
    bool ready = false;       // the key-side counter of `wave` has been seen at its target
    uint64_t next_poll = 0;   // the counter is polled at most once per kPollNs (a poll costs a round trip to L2)
    static constexpr uint64_t kPollNs = 1500;
    // One attempt, called while the warp has nothing else to do.  Returns true if it made progress.
    __device__ __noinline__ bool attempt(const StreamArgs& s, int lane)
    {
        if (wave >= s.waves || wave >= published) return false;
        if (!ready) {
            const uint64_t now = globaltimer_ns();
            if (__all_sync(0xffffffffu, now < next_poll)) return false;
            uint32_t r = 0;
            if (lane == 0) r = counter_reached(s.cnt + wave, s.kdone_target[wave]) ? 1u : 0u;
            if (!__shfl_sync(0xffffffffu, r, 0)) {
                next_poll = now + kPollNs;
                return false;
            }
            ready = true;
#ifdef LINATTN_TRACE
            if (s.trace && lane == 0 && ((threadIdx.x >> 5) & 3) == 0)
                s.trace[(((size_t)blockIdx.x * 4 + 3) * kTraceTiles + 52 + wave) * 4 + 1] = (long long)globaltimer_ns();
#endif
        }
        const int heads = (wave == 0 ? s.gsplit : s.G) - (wave == 0 ? 0 : s.gsplit);
        const int total = heads * kQuadsPerHead;
        const int nwarps = (int)gridDim.x * 4;
        const int gw = (int)blockIdx.x * 4 + ((threadIdx.x >> 5) & 3);
        const long long y = ((long long)step * nwarps + gw) * 32 + lane;   // two lanes per item
#ifdef LINATTN_TRACE
        if (s.trace && lane == 0 && (gw & 3) == 0 && step < 2)
            s.trace[(((size_t)blockIdx.x * 4 + 3) * kTraceTiles + 48 + wave * 2 + step) * 4 + 0] = (long long)globaltimer_ns();
#endif
        combine_item(s, wave, (int)(y >> 1), (int)(y & 1), (y >> 1) < total);
#ifdef LINATTN_TRACE
        if (s.trace && lane == 0 && (gw & 3) == 0 && step < 2)
            s.trace[(((size_t)blockIdx.x * 4 + 3) * kTraceTiles + 48 + wave * 2 + step) * 4 + 1] = (long long)globaltimer_ns();
#endif
        ++step;
        if ((long long)step * nwarps * 16 >= total) {
            // this warp's share of the wave is written: publish it
            __threadfence();
            __syncwarp();
            if (lane == 0) atomicAdd(s.cnt + 2 + wave, 1u);
            ++wave;
            step = 0;
            ready = false;
            next_poll = 0;
        }
        return true;
    }
};

// Aux warps: wait (bounded, abortable, warp-uniform) for a barrier of this CTA's pipeline; while it is not
// ready, work on the combine duty.
__device__ __noinline__ bool aux_wait_barrier(uint32_t bar, uint32_t parity, CombineDuty& duty, const StreamArgs& a,
                                              const WaitCtx& wc, uint32_t code)
{
    const int lane = threadIdx.x & 31;
    const uint64_t t0 = globaltimer_ns();
    uint32_t spins = 0;
    for (;;) {
        // mbarrier.try_wait may keep the warp suspended until the phase completes: fine when there is nothing
        // else to do, but with combine work possibly pending the warp has to come back quickly
        const bool duty_open = duty.wave < a.waves && duty.wave < duty.published;
        const bool done = duty_open ? mbar_test_wait(bar, parity) : mbar_try_wait(bar, parity);
        if (__all_sync(0xffffffffu, done)) return true;
        if (duty.attempt(a, lane)) continue;
        if (duty_open) __nanosleep(100);
        if ((++spins & 63u) != 0u) continue;
        uint32_t ab;
        asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(ab) : "r"(wc.abort_smem) : "memory");
        if (__any_sync(0xffffffffu, ab != 0u || globaltimer_ns() - t0 > kWaitLimitNs)) {
            if (lane == 0) {
                atomicOr(wc.err, code);
                asm volatile("st.volatile.shared.u32 [%0], %1;" ::"r"(wc.abort_smem), "r"(1u) : "memory");
            }
            return false;
        }
    }
}

// Producer: wait (bounded, abortable) until a monotonic counter in global memory has reached its target.
__device__ __noinline__ bool wait_counter(const uint32_t* p, uint32_t target, const WaitCtx& wc)
{
    const int lane = threadIdx.x & 31;
    const uint64_t t0 = globaltimer_ns();
    for (;;) {
        uint32_t r = 0;
        if (lane == 0) r = counter_reached(p, target) ? 1u : 0u;
        if (__shfl_sync(0xffffffffu, r, 0)) return true;
        __nanosleep(256);
        uint32_t ab;
        asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(ab) : "r"(wc.abort_smem) : "memory");
        if (__any_sync(0xffffffffu, ab != 0u || globaltimer_ns() - t0 > kWaitLimitNs)) {
            if (lane == 0) {
                atomicOr(wc.err, (uint32_t)kErrGrid);
                asm volatile("st.volatile.shared.u32 [%0], %1;" ::"r"(wc.abort_smem), "r"(1u) : "memory");
            }
            return false;
        }
    }
}

// ======================================================================================================
// The kernel
// ======================================================================================================

__global__ void __launch_bounds__(kThreads, 1)
linattn_stream_tc(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                  const __grid_constant__ CUtensorMap tmWk, const __grid_constant__ CUtensorMap tmQ,
                  const __grid_constant__ CUtensorMap tmO, const __grid_constant__ CUtensorMap tmWq,
                  const __grid_constant__ CUtensorMap tmS, const StreamArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    LA_TRACE_NS(0, 60, 0);
    // ---- set-up: barriers, TMEM, abort word ----
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SmemStream::kBars);
    const uint32_t bar0 = smem_u32(bars);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(&bars[S_NBARS]);
    uint32_t* abort_word = tmem_slot + 1;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    WaitCtx wc;
    wc.err = a.err;
    wc.abort_smem = smem_u32(abort_word);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    if (threadIdx.x == 0) {
        *abort_word = 0u;
        for (int i = 0; i < kSlots; ++i) {
            mbar_init(bar(S_FULL + i), 1);
            mbar_init(bar(S_EMPTY + i), 1);
            mbar_init(bar(S_PHI + i), 8);
            mbar_init(bar(S_OUT + i), 4);
        }
        for (int i = 0; i < 3; ++i) mbar_init(bar(S_AUX + i), 4);
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(S_UFULL + i), 1);
            mbar_init(bar(S_UEMPTY + i), 8);
            mbar_init(bar(S_WFULL + i), 1);
            mbar_init(bar(S_WFREE + i), 1);
            mbar_init(bar(S_ACCFULL + i), 1);
            mbar_init(bar(S_ACCFREE + i), 4);
        }
        mbar_init(bar(S_STATE), 1);
        mbar_init(bar(S_STATEFREE), 1);
        fence_mbar_init();
    }
    if (warp == 9) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    fence_proxy_async_smem();
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem = *tmem_slot;
    LA_TRACE_NS(0, 60, 1);

    auto slot_addr = [&](int sl) { return sbase + (uint32_t)sl * kTileBytes; };
    // bounded, abortable, warp-uniform wait; flips the role's parity bit on success
    auto wait = [&](Parity& par, int b, uint32_t code) -> bool {
        if (!warp_wait(bar(b), par.get(b), wc, code)) return false;
        par.flip(b);
        return true;
    };

    ItemWalk w;
    w.init(a);

    if (warp == 8) {
        // ================= TMA producer =================
        if (lane == 0) {
            tma_prefetch_desc(&tmK);
            tma_prefetch_desc(&tmV);
            tma_prefetch_desc(&tmWk);
            tma_prefetch_desc(&tmQ);
            tma_prefetch_desc(&tmWq);
            tma_prefetch_desc(&tmS);
        }
        Parity par;
        uint32_t used = 0;        // bit s: slot s has held an item; bit 8+b: W buffer b; bit 10: state buffers
        uint32_t aux_prev = 0;    // bit s: the last item in slot s was a key item (its z column sums read the slot)
        uint32_t inflight = 0, inflight_par = 0;   // loads issued on S_FULL+s and the parity of their phase
        uint32_t full_par = 0;    // producer-side count (mod 2) of fills of each slot
        int pend_g = -1, pend_wave = 0;
        bool ok = true;
        // make slot s free for a new item
        auto acquire_slot = [&](int s) -> bool {
            if (used & (1u << s)) {
                if (!wait(par, S_EMPTY + s, kErrProducer)) return false;
                if (aux_prev & (1u << s)) {
                    if (!wait(par, S_AUX + (s >> 1), kErrProducer)) return false;
                    aux_prev &= ~(1u << s);
                }
            }
            used |= 1u << s;
            return true;
        };
        auto note_fill = [&](int s) {
            inflight |= 1u << s;
            inflight_par = (inflight_par & ~(1u << s)) | (full_par & (1u << s));
            full_par ^= 1u << s;
        };
        // S image and z of head pend_g.  They are written by other CTAs with ordinary stores and become
        // readable once the wave's "combined" counter has reached its target.
        auto state_ready = [&]() -> bool {
            uint32_t r = 0;
            if (lane == 0) r = counter_reached(a.cnt + 2 + pend_wave, a.cdone_target[pend_wave]) ? 1u : 0u;
            return __shfl_sync(0xffffffffu, r, 0) != 0;
        };
        auto load_state = [&](bool block) -> bool {   // returns false only on a time-out
            if (!state_ready()) {
                if (!block) return true;
                if (!wait_counter(a.cnt + 2 + pend_wave, a.cdone_target[pend_wave], wc)) return false;
            }
            if (used & (1u << 10)) {
                if (!wait(par, S_STATEFREE, kErrSeg)) return false;
            } else if (used & (1u << kSSlot)) {
                // first query run: slot 5 may still hold the V tile of a key item
                if (!wait(par, S_EMPTY + kSSlot, kErrSeg)) return false;
            }
            used |= 1u << 10;
            if (lane == 0) {
                fence_proxy_async_all();
                mbar_arrive_expect_tx(bar(S_STATE), kTileBytes + kD * 4);
                tma_load_3d(slot_addr(kSSlot), &tmS, bar(S_STATE), 0, 0, pend_g);
                tma_load_3d(slot_addr(kSSlot) + kHalfTileBytes, &tmS, bar(S_STATE), 64, 0, pend_g);
                bulk_load_1d(sbase + SmemStream::kZ, a.state + (size_t)pend_g * kE + kD * kD, kD * 4, bar(S_STATE));
            }
            pend_g = -1;
            return true;
        };
        for (; !w.done() && ok; w.next()) {
            if (w.first()) {
                if (w.is_q && pend_g >= 0 && !load_state(true)) { ok = false; break; }
                const int wb = w.run & 1;
                if (used & (1u << (8 + wb))) {
                    if (!wait(par, S_WFREE + wb, kErrProducer)) { ok = false; break; }
                }
                used |= 1u << (8 + wb);
                if (lane == 0) {
                    const CUtensorMap* tmW = w.is_q ? &tmWq : &tmWk;
                    mbar_arrive_expect_tx(bar(S_WFULL + wb), kWBytes);
                    const uint32_t wdst = sbase + SmemStream::kW + wb * kWBytes;
                    tma_load_3d(wdst, tmW, bar(S_WFULL + wb), 0, 0, w.g % a.H);
                    tma_load_3d(wdst + kWBytes / 2, tmW, bar(S_WFULL + wb), 64, 0, w.g % a.H);
                }
                if (w.is_q) {
                    pend_g = w.g;
                    pend_wave = w.wave();
                    if (!load_state(false)) { ok = false; break; }
                }
            }
            const int s = w.slot();
            if (!w.is_q) {
                if (!acquire_slot(s) || !acquire_slot(s + 1)) { ok = false; break; }
                aux_prev |= 1u << s;
                LA_TRACE(0, w.ki, 0);
                if (lane == 0) {
                    mbar_arrive_expect_tx(bar(S_FULL + s), 2 * kTileBytes);
                    const uint32_t kdst = slot_addr(s), vdst = slot_addr(s + 1);
                    tma_load_3d(kdst, &tmK, bar(S_FULL + s), 0, w.lt * kTile, w.g);
                    tma_load_3d(kdst + kHalfTileBytes, &tmK, bar(S_FULL + s), 64, w.lt * kTile, w.g);
                    tma_load_3d(vdst, &tmV, bar(S_FULL + s), 0, w.lt * kTile, w.g);
                    tma_load_3d(vdst + kHalfTileBytes, &tmV, bar(S_FULL + s), 64, w.lt * kTile, w.g);
                }
                note_fill(s);
            } else {
                if (pend_g >= 0) {
                    // The state is not there yet.  Keep Q tiles moving while slots are free; once the next slot
                    // is still busy its item may itself be waiting for the state, so the state comes first.
                    if (!load_state(false)) { ok = false; break; }
                    if (pend_g >= 0 && (used & (1u << s))) {
                        uint32_t fr = 0;
                        if (lane == 0) fr = mbar_try_wait(bar(S_EMPTY + s), par.get(S_EMPTY + s)) ? 1u : 0u;
                        fr = __shfl_sync(0xffffffffu, fr, 0);
                        if (!fr && !load_state(true)) { ok = false; break; }
                    }
                }
                if (!acquire_slot(s)) { ok = false; break; }
                LA_TRACE(0, 24 + w.qi, 0);
                if (lane == 0) {
                    mbar_arrive_expect_tx(bar(S_FULL + s), kTileBytes);
                    tma_load_3d(slot_addr(s), &tmQ, bar(S_FULL + s), 0, w.lt * kTile, w.g);
                    tma_load_3d(slot_addr(s) + kHalfTileBytes, &tmQ, bar(S_FULL + s), 64, w.lt * kTile, w.g);
                }
                note_fill(s);
            }
        }
        if (ok && pend_g >= 0) ok = load_state(true);
        if (!ok) {
            // unwinding after a time-out: let the copies already in flight land before the CTA exits
            for (int s = 0; s < kSlots; ++s)
                if (inflight & (1u << s)) mbar_wait(bar(S_FULL + s), (inflight_par >> s) & 1u, kWaitLimitNs);
        }
    } else if (warp == 9) {
        // ================= logits MMA issuer: U = X W =================
        Parity par;
        for (; !w.done(); w.next()) {
            const int wb = w.run & 1, ub = w.i & 1, s = w.slot();
            if (w.first() && !wait(par, S_WFULL + wb, kErrMmaLoad)) break;
            if (!wait(par, S_FULL + s, kErrMmaLoad)) break;
            LA_TRACE(1, w.is_q ? 24 + w.qi : w.ki, 0);
            if (w.i >= 2 && !wait(par, S_UEMPTY + ub, kErrMmaU)) break;
            tcgen05_fence_after();
            if (elect_one()) {
                issue_logits_mma(tmem + kTmemU + ub * kM, slot_addr(s), sbase + SmemStream::kW + wb * kWBytes);
                mma_commit(bar(S_UFULL + ub));
                if (w.last()) mma_commit(bar(S_WFREE + wb));
            }
            __syncwarp();
            LA_TRACE(1, w.is_q ? 24 + w.qi : w.ki, 1);
        }
    } else if (warp == 10) {
        // ================= second MMA issuer: S += phi(k)^T V  /  num = phi(q) S =================
        constexpr uint32_t idesc_s = make_idesc_bf16(kD, kD, 1, 1);      // A = phi^T (MN-major), B = V (MN-major)
        constexpr uint32_t idesc_n = make_idesc_bf16(kTile, kD, 0, 0);   // A = phi(q) (K-major), B = S image [c][f] (K-major)
        const uint64_t kmajor = make_desc_sw128(0, 16, 1024);
        const uint64_t mnmajor = make_desc_sw128(0, kHalfTileBytes, 1024);
        Parity par;
        uint32_t acc_used = 0;
        for (; !w.done(); w.next()) {
            const int s = w.slot(), b = w.acc();
            const uint32_t dacc = tmem + kTmemAcc + b * kD;
            if (!w.is_q) {
                if (!wait(par, S_PHI + s, kErrMmaPhi)) break;
                LA_TRACE(1, w.ki, 2);
                const bool first = w.first();
                if (first) {
                    if ((acc_used & (1u << b)) && !wait(par, S_ACCFREE + b, kErrMmaAcc)) break;
                    acc_used |= 1u << b;
                }
                tcgen05_fence_after();
                if (elect_one()) {
                    const uint32_t phi = slot_addr(s), vt = slot_addr(s + 1);
#pragma unroll
                    for (int k = 0; k < kTile / 16; ++k) {
                        const uint64_t da = desc_at(mnmajor, phi + k * 2048);
                        const uint64_t db = desc_at(mnmajor, vt + k * 2048);
                        mma_bf16_ss(dacc, da, db, idesc_s, (first && k == 0) ? 0u : 1u);
                    }
                    mma_commit(bar(S_EMPTY + s));
                    mma_commit(bar(S_EMPTY + s + 1));
                    if (w.last()) mma_commit(bar(S_ACCFULL + b));
                }
                __syncwarp();
                LA_TRACE(1, w.ki, 3);
            } else {
                if (w.first() && !wait(par, S_STATE, kErrSeg)) break;
                if (!wait(par, S_PHI + s, kErrMmaPhi)) break;
                if ((acc_used & (1u << b)) && !wait(par, S_ACCFREE + b, kErrMmaAcc)) break;
                acc_used |= 1u << b;
                LA_TRACE(1, 24 + w.qi, 2);
                tcgen05_fence_after();
                if (elect_one()) {
                    const uint32_t phi = slot_addr(s), simg = slot_addr(kSSlot);
#pragma unroll
                    for (int k = 0; k < kD / 16; ++k) {
                        const uint64_t da = desc_at(kmajor, phi + (k >> 2) * kHalfTileBytes + (k & 3) * 32);
                        const uint64_t db = desc_at(kmajor, simg + (k >> 2) * kHalfTileBytes + (k & 3) * 32);
                        mma_bf16_ss(dacc, da, db, idesc_n, k > 0);
                    }
                    mma_commit(bar(S_ACCFULL + b));
                    if (w.last()) mma_commit(bar(S_STATEFREE));   // this head's S and z may now be replaced
                }
                __syncwarp();
                LA_TRACE(1, 24 + w.qi, 3);
            }
        }
    } else if (warp == 11) {
        // ================= TMA stores of finished output tiles =================
        // Two stores may be in flight: after issuing item j's store the warp waits only until item j-1's
        // store has read its slot, then hands that slot back to the producer.
        if (lane == 0) tma_prefetch_desc(&tmO);
        Parity par;
        int prev_slot = -1;
        for (; !w.done(); w.next()) {
            if (!w.is_q) continue;
            const int s = w.slot();
            if (!wait(par, S_OUT + s, kErrStore)) break;
            if (lane == 0) {
                tma_store_3d(&tmO, slot_addr(s), 0, w.lt * kTile, w.g);
                tma_store_3d(&tmO, slot_addr(s) + kHalfTileBytes, 64, w.lt * kTile, w.g);
                bulk_commit_group();
                bulk_wait_group_read<1>();
                if (prev_slot >= 0) mbar_arrive(bar(S_EMPTY + prev_slot));
            }
            prev_slot = s;
            __syncwarp();
            LA_TRACE(0, 24 + w.qi, 1);
        }
        if (lane == 0) {
            bulk_wait_group_read<0>();
            if (prev_slot >= 0) mbar_arrive(bar(S_EMPTY + prev_slot));
            bulk_wait_group<0>();
        }
    } else if (warp < 8) {
        // ================= feature map (warps 0-7) =================
        const int half = warp >> 2;                       // 0: softmax(+U), 1: softmax(-U)
        const int row = (warp & 3) * 32 + lane;           // token within the tile == TMEM lane
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const float* z_half = reinterpret_cast<const float*>(smem + SmemStream::kZ) + half * kM;
        Parity par;
        for (; !w.done(); w.next()) {
            const int ub = w.i & 1, s = w.slot();
            if (!wait(par, S_UFULL + ub, kErrSoftmaxU)) break;
            if ((warp & 3) == 0) LA_TRACE(2 + half, w.is_q ? 24 + w.qi : w.ki, 0);
            tcgen05_fence_after();
            float u[kM];
            load_logits(tmem + kTmemU + lane_base + ub * kM, u);
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(S_UEMPTY + ub));
            uint8_t* dst = smem + (size_t)s * kTileBytes + half * kHalfTileBytes + row * 128;
            if (w.is_q && w.first() && !wait(par, S_STATE, kErrSeg)) break;   // z of this head
            const float keep = (w.is_q || w.lt * kTile + row < a.n) ? 1.f : 0.f;
            const float den = softmax_half(u, half != 0, keep, w.is_q ? z_half : nullptr, dst, row);
            if (w.is_q) {
                tmem_st_x1(tmem + kTmemDen + lane_base + 2 * (w.qi & 7) + half, __float_as_uint(den));
                tmem_wait_st();
                tcgen05_fence_before();
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(S_PHI + s));
            if ((warp & 3) == 0) LA_TRACE(2 + half, w.is_q ? 24 + w.qi : w.ki, 1);
        }
    } else {
        // ================= aux warps 12-15: z sums and drains (key), epilogue (query), combine in between ======
        const int aw = warp & 3;
        const int row = aw * 32 + lane;
        const uint32_t lane_base = (uint32_t)(aw * 32) << 16;
        const int sw = row & 7;
        Parity par;
        CombineDuty duty;
        bool ok = true;
        // wait on a barrier of this CTA's pipeline; while it is not ready, work on the combine duty
        auto aux_wait = [&](int b, uint32_t code) -> bool {
            if (!aux_wait_barrier(bar(b), par.get(b), duty, a, wc, code)) return false;
            par.flip(b);
            return true;
        };
        auto publish_key_side = [&](int wave) {
            __threadfence();
            __syncwarp();
            if (lane == 0) atomicAdd(a.cnt + wave, 1u);
            duty.published = wave + 1;
#ifdef LINATTN_TRACE
            if (a.trace && lane == 0 && aw == 0)
                a.trace[(((size_t)blockIdx.x * 4 + 3) * kTraceTiles + 52 + wave) * 4 + 0] = (long long)globaltimer_ns();
#endif
        };
        // waves in which this CTA has no key items are "done" from the start
        for (int wv = 0; wv < a.waves; ++wv) {
            WaveGeom wg;
            wg.init(a, wv);
            const longlong2 r = cta_range(wg.T, gridDim.x, blockIdx.x);
            if (r.y <= r.x) publish_key_side(wv);
        }
        float z0 = 0.f, z1 = 0.f, z2 = 0.f, z3 = 0.f;   // features 2*lane, 2*lane+1, 64+2*lane, 64+2*lane+1 over this warp's 32 tokens
        for (; !w.done() && ok; w.next()) {
            const int s = w.slot(), b = w.acc();
            const uint32_t dacc = tmem + kTmemAcc + b * kD + lane_base;
            if (!w.is_q) {
                if (!aux_wait(S_PHI + s, kErrDrain)) { ok = false; break; }
                // column sums of phi(k) over rows [32 aw, 32 aw + 32) of the tile (rows past the end are zero)
                const uint8_t* blk = smem + (size_t)s * kTileBytes;
#pragma unroll 8
                for (int r = 0; r < 32; ++r) {
                    const int rr = aw * 32 + r;
                    const uint32_t off = (uint32_t)rr * 128u + ((((uint32_t)lane >> 2) ^ ((uint32_t)rr & 7u)) << 4) + ((uint32_t)lane & 3u) * 4u;
                    const uint32_t p0 = *reinterpret_cast<const uint32_t*>(blk + off);
                    const uint32_t p1 = *reinterpret_cast<const uint32_t*>(blk + kHalfTileBytes + off);
                    z0 += __uint_as_float(p0 << 16);
                    z1 += __uint_as_float(p0 & 0xffff0000u);
                    z2 += __uint_as_float(p1 << 16);
                    z3 += __uint_as_float(p1 & 0xffff0000u);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(S_AUX + (s >> 1)));
                if (aw == 0) LA_TRACE(3, w.ki, 2);
                if (w.last()) {
                    // end of this CTA's run in head g: accumulator and z go to the partial record
                    if (!aux_wait(S_ACCFULL + b, kErrDrain)) { ok = false; break; }
                    tcgen05_fence_after();
                    WaveGeom wg;
                    wg.init(a, w.wave());
                    float* rec = a.partial + (size_t)(wg.rec_base + (int)blockIdx.x + (w.g - wg.g0)) * kRec;
                    // thread = feature f = row; the record holds S as [c][f], so that the 32 lanes of a warp
                    // write 128 contiguous bytes per column c
                    float* scol = rec + row;
#pragma unroll
                    for (int c0 = 0; c0 < kD; c0 += 32) {
                        uint32_t v[32];
                        tmem_ld_x32(dacc + c0, v);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 32; ++j) scol[(size_t)(c0 + j) * kD] = __uint_as_float(v[j]);
                    }
                    tcgen05_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(S_ACCFREE + b));
                    float* zp = rec + kD * kD + aw * kD;
                    *reinterpret_cast<float2*>(zp + 2 * lane) = make_float2(z0, z1);
                    *reinterpret_cast<float2*>(zp + kM + 2 * lane) = make_float2(z2, z3);
                    z0 = z1 = z2 = z3 = 0.f;
                    if (w.last_key_of_wave()) publish_key_side(w.wave());
                }
            } else {
                if (!aux_wait(S_ACCFULL + b, kErrEpilogue)) { ok = false; break; }
                if (aw == 0) LA_TRACE(3, 24 + w.qi, 2);
                tcgen05_fence_after();
                uint32_t dv[2];
                tmem_ld_x2(tmem + kTmemDen + lane_base + 2 * (w.qi & 7), dv);
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t v[64];
                    tmem_ld_x32(dacc + half * 64, v);
                    tmem_ld_x32(dacc + half * 64 + 32, v + 32);
                    tmem_wait_ld();
                    if (half == 1) {
                        // everything this item needs from TMEM is in registers: release the accumulator
                        tcgen05_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar(S_ACCFREE + b));
                    }
                    const float inv = __fdividef(1.f, __uint_as_float(dv[0]) + __uint_as_float(dv[1]));
                    const f32x2 inv2 = pack2(inv, inv);
                    uint8_t* dst = smem + (size_t)s * kTileBytes + half * kHalfTileBytes + row * 128;
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
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(S_OUT + s));
                if (aw == 0) LA_TRACE(3, 24 + w.qi, 3);
            }
        }
        // whatever is left of the combine duty (CTAs with few or no items get here early)
        if (ok) {
            const uint64_t t0 = globaltimer_ns();
            while (duty.wave < a.waves) {
                if (duty.attempt(a, lane)) continue;
                __nanosleep(256);
                uint32_t ab;
                asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(ab) : "r"(wc.abort_smem) : "memory");
                if (__any_sync(0xffffffffu, ab != 0u || globaltimer_ns() - t0 > kWaitLimitNs)) {
                    if (lane == 0) {
                        atomicOr(a.err, (uint32_t)kErrGrid);
                        asm volatile("st.volatile.shared.u32 [%0], %1;" ::"r"(wc.abort_smem), "r"(1u) : "memory");
                    }
                    break;
                }
            }
        }
    }
    LA_TRACE_NS(0, 61, 2);
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 9) tmem_dealloc(tmem, 512);
    LA_TRACE_NS(0, 61, 3);
}

}  // namespace tc
}  // namespace linattn
