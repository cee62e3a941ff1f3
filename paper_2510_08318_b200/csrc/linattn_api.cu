// C-ABI boundary of the linear-attention library: context, argument checks, kernel dispatch.
// The entry points and their contracts are declared in include/linattn.h.
#include "linattn.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <new>
#include <type_traits>

#include <nvtx3/nvToolsExt.h>   // header-only: the ranges cost a pointer check unless a profiler is attached

#include "simt_kernels.cuh"
#include "simt_backward.cuh"
#include "sm100_kernels.cuh"
#include "sm100_backward.cuh"
#include "tensor_map.hpp"

using namespace linattn;

namespace {

constexpr int kTargetCtas = 296;  // key-side CTAs aimed for: two waves of the 148 SMs
constexpr int kMaxSplits = 512;

// A named range around each entry point's work on the host (validation, tensor maps, launches), for timelines.
struct NvtxRange {
    explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
    NvtxRange(const NvtxRange&) = delete;
    NvtxRange& operator=(const NvtxRange&) = delete;
};

struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) switched = (cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard()
    {
        if (switched) cudaSetDevice(prev);
    }
};

}  // namespace

struct linattn_ctx {
    int device = 0;
    int H = 0, d = 0;
    long long max_B = 0, max_n = 0;
    bool have_map = false;
    // weights, fp32 [H][d][d/2]
    float* Wq = nullptr;
    float* Wk = nullptr;
    // weights for the tensor-core path: bf16 W^T [H][d/2][d] (d = 128 only)
    __nv_bfloat16* Wqt = nullptr;
    __nv_bfloat16* Wkt = nullptr;
    __nv_bfloat16* Wqt_lo = nullptr;   // what the bf16 rounding of fp32 weights leaves, rounded to bf16 again: W = hi + lo
    __nv_bfloat16* Wkt_lo = nullptr;
    bool map_is_bf16 = false;   // the caller supplied bf16 weights: the images above are exact and the lo parts unused
    __nv_bfloat16* s_img = nullptr;  // [max_B*H][128*128] bf16 image of S for the query-side TMA
    __nv_bfloat16* z_img = nullptr;  // [max_B*H][2048] bf16 operand image of z (hi, lo)
    int num_sms = 0;
    bool coop_ok = false;            // device supports cooperative launches
    uint32_t* sync_words = nullptr;  // fused kernel: 1 + 2 * max_B * H counters (exit count, two meeting points per (b,h) pair), zero between launches
    size_t sync_bytes = 0;
    // workspace
    float* partial = nullptr;   // CUDA-core kernels: [partial_slots][d*d + d]; tensor-core kernels: [partial_slots_tc][128*128 + 128]
    long long partial_slots = 0;
    long long partial_slots_tc = 0;
    float* state = nullptr;     // [max_B*H][d*d + d]
    unsigned int* err_word = nullptr;
    // workspace of the backward pass, allocated by the first linattn_backward
    float* bwd_part_state = nullptr;  // [partial_slots][d*d + d]  per-block sums of dS, dz
    float* bwd_part_w = nullptr;      // [partial_slots][d*d/2]    per-block sums of dW
    float* bwd_part_w2 = nullptr;     // the same for dW_k on the tensor-core path (both weight gradients are summed by one launch at the end)
    float* bwd_dstate = nullptr;      // [max_B*H][d*d + d]        dS, dz
    float* bwd_part_dr = nullptr;     // [partial_slots]           per-block sums of dout . (a - o), the terms of Eq. 8's dL/dr
    __nv_bfloat16* bwd_img[3] = {nullptr, nullptr, nullptr};   // tensor-core backward: lo image of S, hi and lo images of dS
    bool bwd_ready = false;           // every allocation above succeeded
    // host-call staging and its pipeline: copies in, compute and copies out run on three streams, one (b,h) at a time
    void* stage[4] = {nullptr, nullptr, nullptr, nullptr};
    size_t stage_bytes = 0;
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t ev_in = nullptr, ev_done = nullptr, ev_start = nullptr;
    // while linattn_forward_host walks over the (b,h) pairs, the launchers see ONE group: head view_head0's weights,
    // the state slots of group view_g0 (view_H == 0: the whole problem, the normal case)
    int view_H = 0, view_head0 = 0;
    long long view_g0 = 0;
    // options
    int opt_splits = 0;
    int opt_path = 0;
    int opt_fuse = 1;
    int opt_layout = 0;   // 0: [B][H][n][d], 1: [B][n][H][d]
    int opt_phi = 0;      // 0: Hedgehog feature map (Eq. 6), 1: ReLU kernel function
    int opt_reuse = 0;    // 1: linattn_backward may take S, z from the forward that just ran on the same k, v
    long long opt_wait_limit_us = 2000000;   // bound of every device-side wait
    int opt_unmet = 0;    // test hook: the fused kernel's meeting points wait for one arrival that never comes
    // which problem the S, z (tensor-core layout, with the bf16 image of S) in the workspace belong to
    struct StateKey {
        const void* k = nullptr;
        const void* v = nullptr;
        int B = 0, n = 0, layout = 0;
        bool valid = false;
        bool has_lo = false;   // the lo image of S (the backward's second operand) was written along with the state
    } state_key;
    // per-kernel timing (LINATTN_OPT_PROFILE)
    static constexpr int kMaxKernels = 8;
    bool profile = false;
    bool prof_pending = false;
    int prof_n = 0;                       // kernels in the forward being timed
    cudaEvent_t prof_ev[kMaxKernels + 1] = {};
    const char* prof_name[kMaxKernels] = {};
    double prof_bytes[kMaxKernels] = {};
    double prof_ms[kMaxKernels] = {};
    long long prof_cnt[kMaxKernels] = {};
    // bookkeeping
    // shared-memory limit raised on this context's device, per kernel family (function attributes are per device)
    enum AttrSlot { kAttrSimtFwd = 0 /* +0..3: (storage type, head dim) */, kAttrSimtBwd = 4 /* +0..3 */, kAttrTcFwd = 8,
                    kAttrTcBwd = 9, kAttrSlots = 10 };
    bool attr_done[kAttrSlots] = {};
    int last_launches = 0;
    int last_B = 0;
    bool state_transposed = false;  // the last forward left S in the workspace as [c][f] (tensor-core kernels) rather than [f][c]
    char err_text[256] = {0};
#ifdef LINATTN_TRACE
    long long* trace = nullptr;  // tuning builds only: device buffer for per-tile timestamps
#endif
};

namespace {

linattn_status cuda_fail(linattn_ctx* c, cudaError_t e, const char* what)
{
    if (c) snprintf(c->err_text, sizeof(c->err_text), "%s: %s", what, cudaGetErrorString(e));
    return LINATTN_ERR_CUDA;
}

#define LA_CUDA(ctx, call)                                         \
    do {                                                           \
        cudaError_t e__ = (call);                                  \
        if (e__ != cudaSuccess) return cuda_fail(ctx, e__, #call); \
    } while (0)

size_t elem_size(linattn_dtype t) { return t == LINATTN_BF16 ? 2 : 4; }

// Element strides of q, k, v, out for the context's layout option.
ActStrides act_strides(const linattn_ctx* c, int n)
{
    const long long d = c->d, H = c->H;
    if (c->opt_layout == 1) return ActStrides{H * d, d, (long long)n * H * d};   // [B][n][H][d]
    return ActStrides{d, (long long)n * d, H * (long long)n * d};                 // [B][H][n][d]
}

int view_heads(const linattn_ctx* c) { return c->view_H ? c->view_H : c->H; }

// Per-kernel timing: events are recorded around every launch of a forward and read back (after a
// wait on the last one) at the start of the next profiled forward or when the figures are queried.
void prof_flush(linattn_ctx* c)
{
    if (!c->prof_pending) return;
    c->prof_pending = false;
    if (cudaEventSynchronize(c->prof_ev[c->prof_n]) != cudaSuccess) {
        cudaGetLastError();
        return;
    }
    for (int i = 0; i < c->prof_n; ++i) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, c->prof_ev[i], c->prof_ev[i + 1]) == cudaSuccess) {
            c->prof_ms[i] += ms;
            c->prof_cnt[i] += 1;
        }
    }
}

void prof_begin(linattn_ctx* c, cudaStream_t st)
{
    if (!c->profile) return;
    prof_flush(c);
    c->prof_n = 0;
    cudaEventRecord(c->prof_ev[0], st);
}

void prof_mark(linattn_ctx* c, cudaStream_t st, const char* name, double alg_bytes)
{
    if (!c->profile || c->prof_n >= linattn_ctx::kMaxKernels) return;
    const int i = c->prof_n++;
    c->prof_name[i] = name;
    c->prof_bytes[i] = alg_bytes;
    cudaEventRecord(c->prof_ev[i + 1], st);
    c->prof_pending = true;
}

// Splits of the token range per (b,h) for the key-side reduction: enough CTAs to fill the GPU,
// never shorter than 256 tokens each; a function of (G, n) only, so results are reproducible.
int choose_splits(long long G, int n, int forced)
{
    long long s = forced > 0 ? forced : (kTargetCtas + G - 1) / G;
    const long long by_len = (n + 255) / 256;
    if (forced <= 0 && s > by_len) s = by_len;
    if (s > n) s = n;
    if (s > kMaxSplits) s = kMaxSplits;
    if (s < 1) s = 1;
    return (int)s;
}

template <typename T, int D>
linattn_status launch_simt(linattn_ctx* c, const void* q, const void* k, const void* v, void* out, int B, int n,
                           cudaStream_t st, const void* mix, float mix_r)
{
    const int Hv = view_heads(c);
    const long long G = (long long)B * Hv;
    const float* Wq = c->Wq + (size_t)c->view_head0 * D * (D / 2);
    const float* Wk = c->Wk + (size_t)c->view_head0 * D * (D / 2);
    float* state = c->state + (size_t)c->view_g0 * (D * D + D);
    int splits = choose_splits(G, n, c->opt_splits);
    // token chunk per split, rounded up to the kernel's 32-token step; drop splits left empty
    int chunk = (n + splits - 1) / splits;
    chunk = (chunk + kSimtTokens - 1) / kSimtTokens * kSimtTokens;
    splits = (n + chunk - 1) / chunk;
    if (G * splits > c->partial_slots) return LINATTN_ERR_WORKSPACE;
    constexpr int E = D * D + D;

    bool& attr_done = c->attr_done[linattn_ctx::kAttrSimtFwd + (sizeof(T) == 2 ? 2 : 0) + (D == 128 ? 1 : 0)];
    if (!attr_done) {
        LA_CUDA(c, cudaFuncSetAttribute(kside_simt<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)kside_simt_smem<D>()));
        LA_CUDA(c, cudaFuncSetAttribute(qside_simt<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)qside_simt_smem<D>()));
        attr_done = true;
    }
    const double side_bytes = 2.0 * (double)G * n * D * sizeof(T);  // K+V read, or Q read + O written
    prof_begin(c, st);
    kside_simt<T, D><<<dim3(splits, (unsigned)G), kSimtThreads, kside_simt_smem<D>(), st>>>(
        (const T*)k, (const T*)v, Wk, c->partial, Hv, n, chunk, act_strides(c, n), c->opt_phi);
    LA_CUDA(c, cudaGetLastError());
    prof_mark(c, st, "kside_simt", side_bytes);
    combine_state<<<dim3((E + 255) / 256, (unsigned)G), 256, 0, st>>>(c->partial, state, splits, E);
    LA_CUDA(c, cudaGetLastError());
    prof_mark(c, st, "combine_state", 0.0);
    const int nchunks = (n + kSimtTokens - 1) / kSimtTokens;
    long long per_group = (2LL * 148 + G - 1) / G;
    if (per_group > nchunks) per_group = nchunks;
    if (per_group < 1) per_group = 1;
    qside_simt<T, D><<<dim3((unsigned)per_group, (unsigned)G), kSimtThreads, qside_simt_smem<D>(), st>>>(
        (const T*)q, Wq, state, (T*)out, Hv, n, (const T*)mix, mix_r, act_strides(c, n), c->opt_phi);
    LA_CUDA(c, cudaGetLastError());
    prof_mark(c, st, "qside_simt", side_bytes);
    c->last_launches = 3;
    return LINATTN_OK;
}

// Gradients on the CUDA-core kernels: S, z as in the forward, then the query side (dq, dS, dz, dW_q), then the key
// side (dk, dv, dW_k).
// What Eq. 8 adds to a backward call (all unused for the plain operator: lin_scale = 1, the rest null).
struct MixGrad {
    const void* a = nullptr;   // output of the softmax branch
    float lin_scale = 1.f;     // 1 - r^: factor of the gradient that reaches the linear branch
    int r_in_range = 0;        // 0 <= r <= 1: the clip passes the gradient of r
    float* dr = nullptr;       // device, one float
};

template <typename T, int D>
linattn_status launch_backward_simt(linattn_ctx* c, const void* q, const void* k, const void* v, const void* dout, void* dq,
                                    void* dk, void* dv, float* dWq, float* dWk, int per_head, int B, int n, cudaStream_t st,
                                    const MixGrad& mg)
{
    const long long G = (long long)B * c->H;
    int splits = choose_splits(G, n, c->opt_splits);
    int chunk = (n + splits - 1) / splits;
    chunk = (chunk + kSimtTokens - 1) / kSimtTokens * kSimtTokens;
    splits = (n + chunk - 1) / chunk;
    const int nchunks = (n + kSimtTokens - 1) / kSimtTokens;
    long long blocks = (kTargetCtas + G - 1) / G;   // blocks per (b,h) of the two gradient kernels
    if (blocks > nchunks) blocks = nchunks;
    if (G * splits > c->partial_slots || G * blocks > c->partial_slots) return LINATTN_ERR_WORKSPACE;
    constexpr int E = D * D + D, DM = D * (D / 2);

    bool& attr_done = c->attr_done[linattn_ctx::kAttrSimtBwd + (sizeof(T) == 2 ? 2 : 0) + (D == 128 ? 1 : 0)];
    if (!attr_done) {
        LA_CUDA(c, cudaFuncSetAttribute(kside_simt<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kside_simt_smem<D>()));
        LA_CUDA(c, cudaFuncSetAttribute(qside_bwd<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bwd_smem<D>()));
        LA_CUDA(c, cudaFuncSetAttribute(kside_bwd<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bwd_smem<D>()));
        attr_done = true;
    }
    const ActStrides as = act_strides(c, n);
    const double tensor_bytes = (double)G * n * D * sizeof(T);
    const dim3 grid((unsigned)blocks, (unsigned)G);
    prof_begin(c, st);
    const int relu = c->opt_phi;
    kside_simt<T, D><<<dim3(splits, (unsigned)G), kSimtThreads, kside_simt_smem<D>(), st>>>(
        (const T*)k, (const T*)v, c->Wk, c->partial, c->H, n, chunk, as, relu);
    LA_CUDA(c, cudaGetLastError());
    prof_mark(c, st, "kside_simt", 2.0 * tensor_bytes);
    combine_state<<<dim3((E + 255) / 256, (unsigned)G), 256, 0, st>>>(c->partial, c->state, splits, E);
    LA_CUDA(c, cudaGetLastError());
    prof_mark(c, st, "combine_state", 0.0);
    qside_bwd<T, D><<<grid, kSimtThreads, bwd_smem<D>(), st>>>((const T*)q, (const T*)dout, c->Wq, c->state, (T*)dq,
                                                              c->bwd_part_state, c->bwd_part_w, c->H, n, as, relu, (const T*)mg.a,
                                                              mg.lin_scale, mg.dr ? c->bwd_part_dr : nullptr);
    LA_CUDA(c, cudaGetLastError());
    prof_mark(c, st, "qside_bwd", 3.0 * tensor_bytes);
    int launches = 5;
    combine_state<<<dim3((E + 255) / 256, (unsigned)G), 256, 0, st>>>(c->bwd_part_state, c->bwd_dstate, (int)blocks, E);
    LA_CUDA(c, cudaGetLastError());
    const dim3 wgrid((DM + 255) / 256, per_head ? (unsigned)c->H : 1u);
    if (!relu) {   // the ReLU kernel function has no weights
        combine_wgrad<<<wgrid, 256, 0, st>>>(c->bwd_part_w, dWq, (int)blocks, (int)G, c->H, DM, per_head);
        LA_CUDA(c, cudaGetLastError());
        ++launches;
    }
    if (mg.dr) {
        combine_dr<<<1, 32, 0, st>>>(c->bwd_part_dr, (int)(G * blocks), mg.r_in_range, mg.dr);
        LA_CUDA(c, cudaGetLastError());
        ++launches;
    }
    prof_mark(c, st, "combine_dstate_dWq", 0.0);
    kside_bwd<T, D><<<grid, kSimtThreads, bwd_smem<D>(), st>>>((const T*)k, (const T*)v, c->Wk, c->bwd_dstate, (T*)dk, (T*)dv,
                                                              c->bwd_part_w, c->H, n, as, relu);
    LA_CUDA(c, cudaGetLastError());
    prof_mark(c, st, "kside_bwd", 4.0 * tensor_bytes);
    if (!relu) {
        combine_wgrad<<<wgrid, 256, 0, st>>>(c->bwd_part_w, dWk, (int)blocks, (int)G, c->H, DM, per_head);
        LA_CUDA(c, cudaGetLastError());
        ++launches;
    }
    prof_mark(c, st, "combine_dWk", 0.0);
    c->last_launches = launches;
    return LINATTN_OK;
}

// Persistent CTAs of the tensor-core kernels for G (b,h) pairs of T tiles in all: one per SM, except that when (almost)
// all SMs can be used with the SAME number of CTAs per (b,h) pair, that split is taken: then no CTA's run of tiles
// crosses into another pair, so there is one partial record per CTA, one load of S, z and the weights per CTA, and
// the combine sums the same number of records for every pair (measured at B=1, H=12, n=32760: 144 CTAs 82.2 us, 148
// CTAs 84.7 us; with 40 pairs the aligned split would leave 28 SMs idle and loses).  A function of (G, T, #SMs) only.
long long choose_ctas(const linattn_ctx* c, long long G, long long T)
{
    if (T <= c->num_sms) return T;
    const long long per_pair = c->num_sms / G;
    if (per_pair >= 1 && G * per_pair * 100 >= 95LL * c->num_sms) return G * per_pair;
    return c->num_sms;
}

// Tensor-core path: bf16, d = 128, or d = 64 with the heads taken two at a time (the kernels' kPair variant: a pair of
// heads is one 128-feature unit of work with block-diagonal weights and state).
linattn_status launch_tc(linattn_ctx* c, const void* q, const void* k, const void* v, void* out, int B, int n,
                         cudaStream_t st, const void* mix, float mix_r, bool state_only = false)
{
    using namespace linattn::tc;
    const int Hv = view_heads(c);
    const int pair = (c->d == 64) ? 1 : 0;
    const long long heads = (long long)B * Hv;
    const long long G = pair ? (heads + 1) / 2 : heads;   // units of work
    const long long Tn = ((long long)n + kTile - 1) / kTile;
    const long long T = G * Tn;
    long long Pq = choose_ctas(c, G, T);
    long long Pk = Pq;
    if (c->opt_splits > 0) {
        Pk = G * c->opt_splits;
        if (Pk > T) Pk = T;
    }
    if (Pk + G > c->partial_slots_tc) return LINATTN_ERR_WORKSPACE;

    CUtensorMap tmK, tmV, tmQ, tmO, tmWk, tmWq, tmWklo, tmWqlo, tmS, tmA;   // tmA: the softmax branch's output (mixed attention), else a copy of tmQ
    const ActStrides as = act_strides(c, n);
    const int layout = c->opt_layout;
    auto act_map = [&](CUtensorMap* m, const void* base, uint32_t box_rows = kTile) {
        if (layout == 0) return make_tmap_bf16_3d(m, base, (uint64_t)c->d, (uint64_t)n, (uint64_t)heads, box_rows);
        return make_tmap_bf16_act(m, base, (uint64_t)c->d, (uint64_t)n, (uint64_t)Hv, (uint64_t)B, (uint64_t)as.token * 2,
                                  (uint64_t)as.head * 2, (uint64_t)as.batch * 2, box_rows);
    };
    // V is fetched in half tiles (the key side's V ring), everything else in whole tiles
    const bool ok = act_map(&tmK, k) && act_map(&tmV, v, kTile / 2) && act_map(&tmQ, q) && act_map(&tmO, out) && act_map(&tmA, mix ? mix : q) &&
                    make_tmap_bf16_3d(&tmWk, c->Wkt + (size_t)c->view_head0 * kD * kM, kD, kM, (uint64_t)Hv, kM) &&
                    make_tmap_bf16_3d(&tmWq, c->Wqt + (size_t)c->view_head0 * kD * kM, kD, kM, (uint64_t)Hv, kM) &&
                    make_tmap_bf16_3d(&tmWklo, c->Wkt_lo + (size_t)c->view_head0 * kD * kM, kD, kM, (uint64_t)Hv, kM) &&
                    make_tmap_bf16_3d(&tmWqlo, c->Wqt_lo + (size_t)c->view_head0 * kD * kM, kD, kM, (uint64_t)Hv, kM) &&
                    make_tmap_bf16_3d(&tmS, c->s_img + (size_t)c->view_g0 * kD * kD, kD, kD, (uint64_t)G, kTile);
    if (!ok) {
        snprintf(c->err_text, sizeof(c->err_text), "cuTensorMapEncodeTiled failed");
        return LINATTN_ERR_CUDA;
    }
    // one instantiation per (mixed attention or not, memory layout, kernel function, heads singly or in pairs, weights exact
    // in bf16 or split into hi + lo); the ReLU kernel function has no weights, so it has no split variant
#define LA_BY_SPLIT(K, ...) {(const void*)K<__VA_ARGS__, 0>, (const void*)K<__VA_ARGS__, 1>}
#define LA_NO_SPLIT(K, ...) {(const void*)K<__VA_ARGS__, 0>, nullptr}
#define LA_BY_PHI(K, ...) {{LA_BY_SPLIT(K, __VA_ARGS__, 0, 0), LA_BY_SPLIT(K, __VA_ARGS__, 0, 1)}, {LA_NO_SPLIT(K, __VA_ARGS__, 1, 0), LA_NO_SPLIT(K, __VA_ARGS__, 1, 1)}}
    // indices: [mixed][layout][kernel function][pair][split]
    static const void* const k_fused[2][2][2][2][2] = {{LA_BY_PHI(linattn_fused_tc, false, 0), LA_BY_PHI(linattn_fused_tc, false, 1)},
                                                       {LA_BY_PHI(linattn_fused_tc, true, 0), LA_BY_PHI(linattn_fused_tc, true, 1)}};
    static const void* const k_qside[2][2][2][2][2] = {{LA_BY_PHI(qside_tc, false, 0), LA_BY_PHI(qside_tc, false, 1)},
                                                       {LA_BY_PHI(qside_tc, true, 0), LA_BY_PHI(qside_tc, true, 1)}};
    static const void* const k_kside[2][2][2][2] = {LA_BY_PHI(kside_tc, 0), LA_BY_PHI(kside_tc, 1)};
#undef LA_BY_PHI
#undef LA_NO_SPLIT
#undef LA_BY_SPLIT
    const int phi = c->opt_phi;
    const int split = (phi == 0 && !c->map_is_bf16) ? 1 : 0;
    bool& attr_done = c->attr_done[linattn_ctx::kAttrTcFwd];
    if (!attr_done) {
        for (int i = 0; i < 2; ++i)
            for (int p = 0; p < 2; ++p)
                for (int pr = 0; pr < 2; ++pr)
                    for (int sp = 0; sp < 2 - p; ++sp) {
                        LA_CUDA(c, cudaFuncSetAttribute(k_kside[i][p][pr][sp], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Smem::kTotal));
                        for (int j = 0; j < 2; ++j) {
                            LA_CUDA(c, cudaFuncSetAttribute(k_fused[i][j][p][pr][sp], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Smem::kTotal));
                            LA_CUDA(c, cudaFuncSetAttribute(k_qside[i][j][p][pr][sp], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Smem::kTotal));
                        }
                    }
        attr_done = true;
    }
    const double side_bytes = 2.0 * (double)heads * n * c->d * 2;
    Args a{};
    a.partial = c->partial;
    a.state = c->state + (size_t)c->view_g0 * ((size_t)c->d * c->d + c->d);   // one record per head (per pair of heads only inside the kernels)
    a.s_img = c->s_img + (size_t)c->view_g0 * kD * kD;
    // the backward's tensor-core kernels (d = 128) read S as a bf16 hi + lo pair: the lo image is written along with the
    // state when this call is the backward's own, or when the backward may take the state over from this forward
    a.s_img_lo = (!pair && c->bwd_img[0] && c->view_H == 0 && (state_only || c->opt_reuse)) ? c->bwd_img[0] : nullptr;
    a.z_img = c->z_img + (size_t)c->view_g0 * (kZBlkBytes / 2);
    a.err = c->err_word;
    a.sync = c->sync_words;
    a.mix_src = (const __nv_bfloat16*)mix;
    a.mix_r = mix_r;
    a.str_token = as.token;
    a.str_head = as.head;
    a.str_batch = as.batch;
    a.n = n;
    a.H = Hv;
    a.G = (int)G;
    a.heads_total = (int)heads;
    a.tiles_per_head = (int)Tn;
    a.total_tiles = T;
#ifdef LINATTN_TRACE
    a.trace = c->trace;
#endif
    a.wait_limit_us = (uint32_t)c->opt_wait_limit_us;
    a.arrive_extra = c->opt_unmet == 1 ? 1u : 0u;
    prof_begin(c, st);
    if (c->opt_fuse && c->coop_ok && Pk == Pq && !state_only) {
        // one cooperative launch: key side, per-head meeting point, combine, per-head meeting point, query side.  Its
        // counters are zero between launches (the kernel clears them on its way out), so nothing here depends on
        // earlier launches and the launch may be recorded in a CUDA graph.
        void* params[] = {&tmK, &tmV, &tmWk, &tmWklo, &tmQ, &tmO, &tmWq, &tmWqlo, &tmS, &tmA, &a};
        const cudaError_t le = cudaLaunchCooperativeKernel(k_fused[mix ? 1 : 0][layout][phi][pair][split], dim3((unsigned)Pq), dim3(kThreads),
                                                           params, Smem::kTotal, st);
        if (le == cudaSuccess) {
            prof_mark(c, st, "linattn_fused_tc", 2.0 * side_bytes);
            c->last_launches = 1;
            return LINATTN_OK;
        }
        if (le != cudaErrorCooperativeLaunchTooLarge) return cuda_fail(c, le, "cudaLaunchCooperativeKernel");
        // Not all CTAs can be resident at once (part of the GPU is taken, e.g. MIG or MPS limits): nothing was
        // launched; use the three-launch form from now on, which needs no co-residency.
        cudaGetLastError();
        c->coop_ok = false;
    }
    {
        void* kp[] = {&tmK, &tmV, &tmWk, &tmWklo, &a};
        LA_CUDA(c, cudaLaunchKernel(k_kside[layout][phi][pair][split], dim3((unsigned)Pk), dim3(kThreads), kp, Smem::kTotal, st));
    }
    LA_CUDA(c, cudaGetLastError());
    prof_mark(c, st, "kside_tc", side_bytes);
    if (pair) combine_tc<1><<<dim3((kE / 4 + 255) / 256, (unsigned)G), 256, 0, st>>>(a, Pk);
    else combine_tc<0><<<dim3((kE / 4 + 255) / 256, (unsigned)G), 256, 0, st>>>(a, Pk);
    LA_CUDA(c, cudaGetLastError());
    prof_mark(c, st, "combine_tc", 0.0);
    if (state_only) {   // the backward pass wants S and z only
        c->last_launches = 2;
        return LINATTN_OK;
    }
    {
        void* qp[] = {&tmQ, &tmO, &tmWq, &tmWqlo, &tmS, &tmA, &a};
        LA_CUDA(c, cudaLaunchKernel(k_qside[mix ? 1 : 0][layout][phi][pair][split], dim3((unsigned)Pq), dim3(kThreads), qp, Smem::kTotal, st));
    }
    LA_CUDA(c, cudaGetLastError());
    prof_mark(c, st, "qside_tc", side_bytes);
    c->last_launches = 3;
    return LINATTN_OK;
}

// Gradients on the tensor-core kernels (bf16, d = 128, bf16 feature-map weights): S, z by the forward's key-side
// kernels, then the query side (dq; dS, dz, dW_q records), the combines, and the key side (dk, dv; dW_k records).
linattn_status launch_backward_tc(linattn_ctx* c, const void* q, const void* k, const void* v, const void* dout, void* dq,
                                  void* dk, void* dv, float* dWq, float* dWk, int per_head, int B, int n, cudaStream_t st,
                                  const MixGrad& mg)
{
    using namespace linattn::tc;
    const long long G = (long long)B * c->H;
    const long long Tn = ((long long)n + kTile - 1) / kTile;
    const long long T = G * Tn;
    const long long P = c->num_sms < T ? c->num_sms : T;   // these kernels are bound by per-tile latency, not bandwidth: every SM counts
    if (P + G > c->partial_slots_tc) return LINATTN_ERR_WORKSPACE;
    // forward state (S as [c][f], z) and the hi image of S: left by the forward that just ran on these k, v (if the
    // caller allows it), else recomputed; q and out are not touched by the first two kernels of the forward
    const linattn_ctx::StateKey& sk = c->state_key;
    const bool reuse = c->opt_reuse && sk.valid && sk.k == k && sk.v == v && sk.B == B && sk.n == n && sk.layout == c->opt_layout;
    int launches = 4;   // qside_bwd_tc, combine of dS and dz, kside_bwd_tc, combine of both weight gradients
    bool need_lo = false;
    if (reuse) {
        prof_begin(c, st);
        need_lo = !sk.has_lo;
    } else {
        c->state_key.valid = false;
        const linattn_status s = launch_tc(c, k, k, v, dk, B, n, st, nullptr, 0.f, true);   // writes the lo image of S too
        if (s != LINATTN_OK) return s;
        c->state_key = {k, v, B, n, c->opt_layout, true, true};
        launches = 6;
    }

    const ActStrides as = act_strides(c, n);
    const int layout = c->opt_layout;
    auto act_map = [&](CUtensorMap* m, const void* base) {
        if (layout == 0) return make_tmap_bf16_3d(m, base, kD, (uint64_t)n, (uint64_t)G, kTile);
        return make_tmap_bf16_act(m, base, kD, (uint64_t)n, (uint64_t)c->H, (uint64_t)B, (uint64_t)as.token * 2,
                                  (uint64_t)as.head * 2, (uint64_t)as.batch * 2, kTile);
    };
    auto img_map = [&](CUtensorMap* m, const void* base) { return make_tmap_bf16_3d(m, base, kD, kD, (uint64_t)G, kTile); };
    CUtensorMap tmQ, tmG, tmDQ, tmK, tmV, tmDK, tmDV, tmWq, tmWk, tmShi, tmSlo, tmDShi, tmDSlo;
    const bool ok = act_map(&tmQ, q) && act_map(&tmG, dout) && act_map(&tmDQ, dq) && act_map(&tmK, k) && act_map(&tmV, v) &&
                    act_map(&tmDK, dk) && act_map(&tmDV, dv) &&
                    make_tmap_bf16_3d(&tmWq, c->Wqt, kD, kM, (uint64_t)c->H, kM) &&
                    make_tmap_bf16_3d(&tmWk, c->Wkt, kD, kM, (uint64_t)c->H, kM) && img_map(&tmShi, c->s_img) &&
                    img_map(&tmSlo, c->bwd_img[0]) && img_map(&tmDShi, c->bwd_img[1]) && img_map(&tmDSlo, c->bwd_img[2]);
    if (!ok) {
        snprintf(c->err_text, sizeof(c->err_text), "cuTensorMapEncodeTiled failed");
        return LINATTN_ERR_CUDA;
    }
    const void* k_q[2][2] = {{(const void*)qside_bwd_tc<0, 0>, (const void*)qside_bwd_tc<0, 1>},
                             {(const void*)qside_bwd_tc<1, 0>, (const void*)qside_bwd_tc<1, 1>}};   // [layout][Eq. 8 terms]
    const void* k_k[2] = {(const void*)kside_bwd_tc<0>, (const void*)kside_bwd_tc<1>};
    bool& attr_done = c->attr_done[linattn_ctx::kAttrTcBwd];
    if (!attr_done) {
        for (int i = 0; i < 2; ++i) {
            for (int j = 0; j < 2; ++j) LA_CUDA(c, cudaFuncSetAttribute(k_q[i][j], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBwdSmemQ));
            LA_CUDA(c, cudaFuncSetAttribute(k_k[i], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBwdSmemK));
        }
        attr_done = true;
    }
    const double tensor_bytes = (double)G * n * kD * 2;
    BwdArgs a{};
    a.part_state = c->bwd_part_state;
    a.part_w = c->bwd_part_w;
    a.state = c->state;
    a.err = c->err_word;
    a.mix_a = (const __nv_bfloat16*)mg.a;
    a.part_dr = c->bwd_part_dr;
    a.lin_scale = mg.lin_scale;
    a.str_token = as.token;
    a.str_head = as.head;
    a.str_batch = as.batch;
    a.n = n;
    a.H = c->H;
    a.G = (int)G;
    a.tiles_per_head = (int)Tn;
    a.total_tiles = T;
    a.wait_limit_us = (uint32_t)c->opt_wait_limit_us;
    a.test_unmet = c->opt_unmet == 2 ? 1 : 0;
#ifdef LINATTN_TRACE
    a.trace = c->trace;
#endif
    const dim3 wgrid(kWRec / 256, per_head ? (unsigned)c->H : 1u);
    if (need_lo) {   // the state was taken over from a forward that ran before the backward's workspace existed
        hilo_images<<<dim3(kD * kD / 256, (unsigned)G), 256, 0, st>>>(c->state, nullptr, c->bwd_img[0]);
        LA_CUDA(c, cudaGetLastError());
        c->state_key.has_lo = true;
        ++launches;
    }
    {
        void* p[] = {&tmQ, &tmG, &tmDQ, &tmWq, &tmShi, &tmSlo, &a};
        LA_CUDA(c, cudaLaunchKernel(k_q[layout][mg.dr ? 1 : 0], dim3((unsigned)P), dim3(kBwdThreads), p, kBwdSmemQ, st));
    }
    prof_mark(c, st, "qside_bwd_tc", (mg.dr ? 4.0 : 3.0) * tensor_bytes);
    if (mg.dr) {
        combine_dr<<<1, 32, 0, st>>>(c->bwd_part_dr, (int)P, mg.r_in_range, mg.dr);
        LA_CUDA(c, cudaGetLastError());
        ++launches;
    }
    combine_slots_hilo<<<dim3((kE + 255) / 256, (unsigned)G), 256, 0, st>>>(c->bwd_part_state, c->bwd_dstate, c->bwd_img[1], c->bwd_img[2],
                                                                           (int)Tn, T, P);
    LA_CUDA(c, cudaGetLastError());
    prof_mark(c, st, "combine_dstate", 0.0);
    a.state = c->bwd_dstate;
    a.test_unmet = c->opt_unmet == 3 ? 1 : 0;
    a.part_w = c->bwd_part_w2;   // dW_k's records; dW_q's stay in part_w until both are summed at the end
    {
        void* p[] = {&tmK, &tmV, &tmDK, &tmDV, &tmWk, &tmDShi, &tmDSlo, &a};
        LA_CUDA(c, cudaLaunchKernel(k_k[layout], dim3((unsigned)P), dim3(kBwdThreads), p, kBwdSmemK, st));
    }
    prof_mark(c, st, "kside_bwd_tc", 4.0 * tensor_bytes);
    combine_wgrad_slots2<<<dim3(wgrid.x, wgrid.y, 2), 256, 0, st>>>(c->bwd_part_w, c->bwd_part_w2, dWq, dWk, (int)G, c->H, per_head, (int)Tn, T, P);
    LA_CUDA(c, cudaGetLastError());
    prof_mark(c, st, "combine_dWq_dWk", 0.0);
    c->last_launches = launches;
    return LINATTN_OK;
}

bool misaligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

bool overlaps(const void* a, const void* b, size_t bytes)
{
    const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
    return x < y + bytes && y < x + bytes;
}

linattn_status check_forward_args(linattn_ctx* c, const void* q, const void* k, const void* v, void* out, int B,
                                  int H, int n, int d, linattn_dtype dtype)
{
    if (!c || !q || !k || !v || !out) return LINATTN_ERR_INVALID_ARG;
    if (dtype != LINATTN_F32 && dtype != LINATTN_BF16) return LINATTN_ERR_UNSUPPORTED;
    if (d != 64 && d != 128) return LINATTN_ERR_UNSUPPORTED;
    if (H != c->H || d != c->d) return LINATTN_ERR_INVALID_ARG;
    if (B < 1 || n < 1) return LINATTN_ERR_INVALID_ARG;
    if (B > c->max_B || n > c->max_n) return LINATTN_ERR_WORKSPACE;
    if (!c->have_map && c->opt_phi == 0) return LINATTN_ERR_NO_FEATURE_MAP;   // the ReLU kernel function has no weights
    return LINATTN_OK;
}

}  // namespace

extern "C" {

const char* linattn_status_string(linattn_status s)
{
    switch (s) {
        case LINATTN_OK: return "ok";
        case LINATTN_ERR_INVALID_ARG: return "invalid argument";
        case LINATTN_ERR_UNSUPPORTED: return "unsupported head dimension, dtype or device";
        case LINATTN_ERR_NO_FEATURE_MAP: return "feature map not set";
        case LINATTN_ERR_WORKSPACE: return "request exceeds the workspace reserved at create";
        case LINATTN_ERR_CUDA: return "CUDA error";
        case LINATTN_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

linattn_status linattn_create(linattn_ctx** out_ctx, int device, int H, int d, long long max_B, long long max_n)
{
    if (!out_ctx || H < 1 || max_B < 1 || max_n < 1 || device < 0) return LINATTN_ERR_INVALID_ARG;
    if (max_n > 0x7fffffffLL || max_B * H > 65535) return LINATTN_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return LINATTN_ERR_UNSUPPORTED;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device >= ndev) {
        cudaGetLastError();
        return LINATTN_ERR_CUDA;
    }
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess)
        return LINATTN_ERR_CUDA;
    if (major != 10) return LINATTN_ERR_UNSUPPORTED;

    linattn_ctx* c = new (std::nothrow) linattn_ctx();
    if (!c) return LINATTN_ERR_INVALID_ARG;
    c->device = device;
    c->H = H;
    c->d = d;
    c->max_B = max_B;
    c->max_n = max_n;
    DeviceGuard guard(device);
    const size_t E = (size_t)d * d + d;
    const size_t wbytes = sizeof(float) * (size_t)H * d * (d / 2);
    const long long G = max_B * H;
    // The tensor-core kernels work on 128-feature units (one head of dimension 128, or a pair of heads of dimension 64:
    // at most G units either way) with records of 128 * 128 + 128 floats, one per persistent CTA and unit it touches.
    c->partial_slots = kTargetCtas + G;
    c->partial_slots_tc = kTargetCtas + G;
    const size_t simt_bytes = sizeof(float) * E * (size_t)c->partial_slots;
    const size_t tc_bytes = sizeof(float) * (size_t)linattn::tc::kE * (size_t)c->partial_slots_tc;
    cudaError_t e = cudaSuccess;
    if (e == cudaSuccess) e = cudaMalloc(&c->Wq, wbytes);
    if (e == cudaSuccess) e = cudaMalloc(&c->Wk, wbytes);
    if (e == cudaSuccess) e = cudaMalloc(&c->partial, simt_bytes > tc_bytes ? simt_bytes : tc_bytes);
    if (e == cudaSuccess) e = cudaMalloc(&c->state, sizeof(float) * E * (size_t)G);
    if (e == cudaSuccess) {
        // weight images W^T [H][64][128] bf16 (d = 64: of each pair of consecutive heads), bf16 image of S and operand image of z per unit
        const size_t wt = sizeof(__nv_bfloat16) * (size_t)H * linattn::tc::kM * linattn::tc::kD;
        e = cudaMalloc(&c->Wqt, wt);
        if (e == cudaSuccess) e = cudaMalloc(&c->Wkt, wt);
        if (e == cudaSuccess) e = cudaMalloc(&c->Wqt_lo, wt);
        if (e == cudaSuccess) e = cudaMalloc(&c->Wkt_lo, wt);
        if (e == cudaSuccess) e = cudaMalloc(&c->s_img, sizeof(__nv_bfloat16) * (size_t)G * linattn::tc::kD * linattn::tc::kD);
        if (e == cudaSuccess) e = cudaMalloc(&c->z_img, (size_t)G * linattn::tc::kZBlkBytes);
        if (e == cudaSuccess) e = cudaMemset(c->z_img, 0, (size_t)G * linattn::tc::kZBlkBytes);
    }
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->num_sms, cudaDevAttrMultiProcessorCount, device);
    if (e == cudaSuccess) {
        int coop = 0;
        e = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, device);
        c->coop_ok = (coop != 0);
    }
    c->sync_bytes = sizeof(uint32_t) * (size_t)(1 + 2 * G);
    if (e == cudaSuccess) e = cudaMalloc(&c->sync_words, c->sync_bytes);
    if (e == cudaSuccess) e = cudaMemset(c->sync_words, 0, c->sync_bytes);
    if (e == cudaSuccess) e = cudaMalloc(&c->err_word, sizeof(unsigned int));
    if (e == cudaSuccess) e = cudaMemset(c->err_word, 0, sizeof(unsigned int));
    if (e != cudaSuccess) {
        cudaGetLastError();
        linattn_destroy(c);
        return LINATTN_ERR_CUDA;
    }
    *out_ctx = c;
    return LINATTN_OK;
}

linattn_status linattn_destroy(linattn_ctx* c)
{
    if (!c) return LINATTN_OK;
    DeviceGuard guard(c->device);
    cudaDeviceSynchronize();
    cudaFree(c->Wq);
    cudaFree(c->Wk);
    cudaFree(c->partial);
    cudaFree(c->state);
    cudaFree(c->err_word);
    cudaFree(c->sync_words);
    cudaFree(c->Wqt);
    cudaFree(c->Wkt);
    cudaFree(c->Wqt_lo);
    cudaFree(c->Wkt_lo);
    cudaFree(c->s_img);
    cudaFree(c->z_img);
    cudaFree(c->bwd_part_state);
    cudaFree(c->bwd_part_w);
    cudaFree(c->bwd_part_w2);
    cudaFree(c->bwd_dstate);
    cudaFree(c->bwd_part_dr);
    for (void* p : c->bwd_img) cudaFree(p);
    for (void* p : c->stage) cudaFree(p);
    if (c->copy_in) cudaStreamDestroy(c->copy_in);
    if (c->copy_out) cudaStreamDestroy(c->copy_out);
    if (c->ev_in) cudaEventDestroy(c->ev_in);
    if (c->ev_done) cudaEventDestroy(c->ev_done);
    if (c->ev_start) cudaEventDestroy(c->ev_start);
    for (cudaEvent_t ev : c->prof_ev)
        if (ev) cudaEventDestroy(ev);
    cudaGetLastError();
    delete c;
    return LINATTN_OK;
}

linattn_status linattn_set_feature_map(linattn_ctx* c, const void* Wq, const void* Wk, int per_head,
                                       linattn_dtype wdtype, void* stream)
{
    NvtxRange range("linattn_set_feature_map");
    if (!c || !Wq || !Wk) return LINATTN_ERR_INVALID_ARG;
    if (wdtype != LINATTN_F32 && wdtype != LINATTN_BF16) return LINATTN_ERR_UNSUPPORTED;
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    const int DM = c->d * (c->d / 2);
    const size_t total = (size_t)c->H * DM;
    const unsigned blocks = (unsigned)((total + 255) / 256);
    if (wdtype == LINATTN_F32) {
        convert_weights<float><<<blocks, 256, 0, st>>>((const float*)Wq, c->Wq, c->H, DM, per_head ? 1 : 0);
        convert_weights<float><<<blocks, 256, 0, st>>>((const float*)Wk, c->Wk, c->H, DM, per_head ? 1 : 0);
    } else {
        convert_weights<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)Wq, c->Wq, c->H, DM, per_head ? 1 : 0);
        convert_weights<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)Wk, c->Wk, c->H, DM, per_head ? 1 : 0);
    }
    {
        // images for the tensor-core kernels: W^T [H][64][128] bf16 (d = 64: of each pair of consecutive heads); fp32 weights
        // are kept as a bf16 hi + lo pair
        const unsigned tb = (unsigned)(((size_t)c->H * tc::kM * tc::kD + 255) / 256);
        const int ph = per_head ? 1 : 0;
        auto images = [&](auto src_q, auto src_k) {
            using T = std::remove_cv_t<std::remove_pointer_t<decltype(src_q)>>;
            for (int lo = 0; lo < (wdtype == LINATTN_F32 ? 2 : 1); ++lo) {
                __nv_bfloat16* dq = lo ? c->Wqt_lo : c->Wqt;
                __nv_bfloat16* dk = lo ? c->Wkt_lo : c->Wkt;
                if (c->d == 64) {
                    tc::pair_weights_bf16<T><<<tb, 256, 0, st>>>(src_q, dq, c->H, ph, lo);
                    tc::pair_weights_bf16<T><<<tb, 256, 0, st>>>(src_k, dk, c->H, ph, lo);
                } else {
                    tc::transpose_weights_bf16<T><<<tb, 256, 0, st>>>(src_q, dq, c->H, ph, lo);
                    tc::transpose_weights_bf16<T><<<tb, 256, 0, st>>>(src_k, dk, c->H, ph, lo);
                }
            }
        };
        if (wdtype == LINATTN_F32) images((const float*)Wq, (const float*)Wk);
        else images((const __nv_bfloat16*)Wq, (const __nv_bfloat16*)Wk);
    }
    LA_CUDA(c, cudaGetLastError());
    c->map_is_bf16 = (wdtype == LINATTN_BF16);
    c->have_map = true;
    c->state_key.valid = false;
    return LINATTN_OK;
}

static linattn_status dispatch_forward(linattn_ctx* c, const void* q, const void* k, const void* v, void* out, const void* mix,
                                       float mix_r, int B, int n, int d, linattn_dtype dtype, cudaStream_t st);

// Shared by linattn_forward (mix == NULL) and linattn_forward_mixed.
static linattn_status forward_impl(linattn_ctx* c, const void* q, const void* k, const void* v, void* out,
                                   const void* mix, float mix_r, int B, int H, int n, int d, linattn_dtype dtype,
                                   void* stream)
{
    NvtxRange range(mix ? "linattn_forward_mixed" : "linattn_forward");
    linattn_status s = check_forward_args(c, q, k, v, out, B, H, n, d, dtype);
    if (s != LINATTN_OK) return s;
    if (misaligned16(q) || misaligned16(k) || misaligned16(v) || misaligned16(out)) return LINATTN_ERR_INVALID_ARG;
    const size_t bytes = (size_t)B * H * n * d * elem_size(dtype);
    if (overlaps(out, q, bytes) || overlaps(out, k, bytes) || overlaps(out, v, bytes)) return LINATTN_ERR_INVALID_ARG;
    if (mix) {
        if (misaligned16(mix)) return LINATTN_ERR_INVALID_ARG;
        if (mix != out && overlaps(out, mix, bytes)) return LINATTN_ERR_INVALID_ARG;  // in place is fine, a partial overlap is not
        if (!(mix_r == mix_r)) return LINATTN_ERR_INVALID_ARG;                         // NaN
        mix_r = mix_r < 0.f ? 0.f : (mix_r > 1.f ? 1.f : mix_r);                       // footnote to Eq. 8: r is clipped into [0, 1]
    }
    DeviceGuard guard(c->device);
    return dispatch_forward(c, q, k, v, out, mix, mix_r, B, n, d, dtype, (cudaStream_t)stream);
}

// Choice of kernels for checked arguments.  The tensor-core kernels cover bf16 activations (head dimension 128, or 64
// with the heads taken in pairs; feature-map weights given in fp32 enter as a bf16 hi + lo pair); fp32 activations run
// on the CUDA-core kernels.
static linattn_status dispatch_forward(linattn_ctx* c, const void* q, const void* k, const void* v, void* out, const void* mix,
                                       float mix_r, int B, int n, int d, linattn_dtype dtype, cudaStream_t st)
{
    const bool tc_ok = (dtype == LINATTN_BF16);   // d = 128, or d = 64 with the heads in pairs; weights of either type
    if (c->opt_path == 2 && !tc_ok) return LINATTN_ERR_UNSUPPORTED;
    c->last_B = B;
    c->state_transposed = tc_ok && c->opt_path != 1;
    c->state_key.valid = false;
    if (c->state_transposed) {
        const linattn_status s = launch_tc(c, q, k, v, out, B, n, st, mix, mix_r);
        if (s == LINATTN_OK && c->opt_phi == 0 && c->view_H == 0 && d == 128)
            c->state_key = {k, v, B, n, c->opt_layout, true, c->opt_reuse && c->bwd_img[0] != nullptr};
        return s;
    }
    if (dtype == LINATTN_BF16) {
        return d == 128 ? launch_simt<__nv_bfloat16, 128>(c, q, k, v, out, B, n, st, mix, mix_r)
                        : launch_simt<__nv_bfloat16, 64>(c, q, k, v, out, B, n, st, mix, mix_r);
    }
    return d == 128 ? launch_simt<float, 128>(c, q, k, v, out, B, n, st, mix, mix_r)
                    : launch_simt<float, 64>(c, q, k, v, out, B, n, st, mix, mix_r);
}

linattn_status linattn_forward(linattn_ctx* c, const void* q, const void* k, const void* v, void* out, int B, int H,
                               int n, int d, linattn_dtype dtype, void* stream)
{
    return forward_impl(c, q, k, v, out, nullptr, 0.f, B, H, n, d, dtype, stream);
}

linattn_status linattn_forward_mixed(linattn_ctx* c, const void* q, const void* k, const void* v,
                                     const void* o_softmax, float r, void* out, int B, int H, int n, int d,
                                     linattn_dtype dtype, void* stream)
{
    if (!o_softmax) return LINATTN_ERR_INVALID_ARG;
    return forward_impl(c, q, k, v, out, o_softmax, r, B, H, n, d, dtype, stream);
}

// Shared by linattn_backward (a == NULL) and linattn_backward_mixed.
static linattn_status backward_impl(linattn_ctx* c, const void* q, const void* k, const void* v, const void* a, float r,
                                    const void* dout, void* dq, void* dk, void* dv, float* dWq, float* dWk, int per_head,
                                    void* d_a, float* dr, int B, int H, int n, int d, linattn_dtype dtype, void* stream)
{
    NvtxRange range(a ? "linattn_backward_mixed" : "linattn_backward");
    if (!dout || !dk || !dv) return LINATTN_ERR_INVALID_ARG;
    const bool relu = c && c->opt_phi != 0;
    if (!relu && (!dWq || !dWk)) return LINATTN_ERR_INVALID_ARG;   // the ReLU kernel function has no weights: its dWq, dWk are ignored
    linattn_status s = check_forward_args(c, q, k, v, dq, B, H, n, d, dtype);
    if (s != LINATTN_OK) return s;
    const void* ins[5] = {q, k, v, dout, a};
    void* outs[4] = {dq, dk, dv, d_a};
    const size_t bytes = (size_t)B * H * n * d * elem_size(dtype);
    for (const void* p : ins)
        if (p && misaligned16(p)) return LINATTN_ERR_INVALID_ARG;
    for (int i = 0; i < 4; ++i) {
        if (!outs[i]) continue;
        if (misaligned16(outs[i])) return LINATTN_ERR_INVALID_ARG;
        for (const void* p : ins)
            if (p && overlaps(outs[i], p, bytes)) return LINATTN_ERR_INVALID_ARG;
        for (int j = 0; j < i; ++j)
            if (outs[j] && overlaps(outs[i], outs[j], bytes)) return LINATTN_ERR_INVALID_ARG;
    }
    if (!relu && (misaligned16(dWq) || misaligned16(dWk) || dWq == dWk)) return LINATTN_ERR_INVALID_ARG;
    MixGrad mg;
    if (a) {
        if (!dr || (reinterpret_cast<uintptr_t>(dr) & 3u) || !(r == r)) return LINATTN_ERR_INVALID_ARG;
        const float rc = r < 0.f ? 0.f : (r > 1.f ? 1.f : r);   // footnote to Eq. 8: r is clipped into [0, 1]
        mg.a = a;
        mg.lin_scale = 1.f - rc;
        mg.r_in_range = (r >= 0.f && r <= 1.f) ? 1 : 0;   // the clip passes r's gradient on the closed interval
        mg.dr = dr;
    }
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    if (!c->bwd_ready) {
        // all or nothing: a failed allocation releases what the earlier ones got, so that the next call starts over
        const size_t E = (size_t)d * d + d, G = (size_t)(c->max_B * c->H);
        cudaError_t e = cudaMalloc(&c->bwd_part_state, sizeof(float) * E * (size_t)c->partial_slots);
        if (e == cudaSuccess) e = cudaMalloc(&c->bwd_part_w, sizeof(float) * (size_t)d * (d / 2) * (size_t)c->partial_slots);
        if (e == cudaSuccess && d == 128) e = cudaMalloc(&c->bwd_part_w2, sizeof(float) * (size_t)d * (d / 2) * (size_t)c->partial_slots);
        if (e == cudaSuccess) e = cudaMalloc(&c->bwd_dstate, sizeof(float) * E * G);
        if (e == cudaSuccess) e = cudaMalloc(&c->bwd_part_dr, sizeof(float) * (size_t)c->partial_slots);
        if (d == 128)
            for (__nv_bfloat16*& p : c->bwd_img)
                if (e == cudaSuccess) e = cudaMalloc(&p, sizeof(__nv_bfloat16) * (size_t)d * d * G);
        if (e != cudaSuccess) {
            cudaGetLastError();
            cudaFree(c->bwd_part_state);
            cudaFree(c->bwd_part_w);
            cudaFree(c->bwd_part_w2);
            cudaFree(c->bwd_dstate);
            cudaFree(c->bwd_part_dr);
            c->bwd_part_state = c->bwd_part_w = c->bwd_part_w2 = c->bwd_dstate = c->bwd_part_dr = nullptr;
            for (__nv_bfloat16*& p : c->bwd_img) {
                cudaFree(p);
                p = nullptr;
            }
            return cuda_fail(c, e, "cudaMalloc (backward workspace)");
        }
        c->bwd_ready = true;
    }
    c->last_B = B;
    const int ph = per_head ? 1 : 0;
    // the gradient that reaches the softmax branch, r^ * dout: element by element, whatever the layout
    if (a && d_a) {
        const size_t count = (size_t)B * H * n * d;
        const unsigned blocks = (unsigned)((count + 256 * 8 - 1) / (256 * 8) < 1184 * 4 ? (count + 256 * 8 - 1) / (256 * 8) : 1184 * 4);
        if (dtype == LINATTN_BF16) scale_copy<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)dout, (__nv_bfloat16*)d_a, count, 1.f - mg.lin_scale);
        else scale_copy<float><<<blocks, 256, 0, st>>>((const float*)dout, (float*)d_a, count, 1.f - mg.lin_scale);
        LA_CUDA(c, cudaGetLastError());
    }
    // tensor-core kernels: Eq. 6 with bf16 weights, bf16 activations, d = 128; everything else on the CUDA cores
    const bool tc_ok = (dtype == LINATTN_BF16 && d == 128 && c->map_is_bf16 && !relu);
    if (c->opt_path == 2 && !tc_ok) return LINATTN_ERR_UNSUPPORTED;
    linattn_status res;
    if (tc_ok && c->opt_path != 1) {
        c->state_transposed = true;
        res = launch_backward_tc(c, q, k, v, dout, dq, dk, dv, dWq, dWk, ph, B, n, st, mg);
    } else {
        c->state_transposed = false;
        c->state_key.valid = false;
        if (dtype == LINATTN_BF16)
            res = d == 128 ? launch_backward_simt<__nv_bfloat16, 128>(c, q, k, v, dout, dq, dk, dv, dWq, dWk, ph, B, n, st, mg)
                           : launch_backward_simt<__nv_bfloat16, 64>(c, q, k, v, dout, dq, dk, dv, dWq, dWk, ph, B, n, st, mg);
        else
            res = d == 128 ? launch_backward_simt<float, 128>(c, q, k, v, dout, dq, dk, dv, dWq, dWk, ph, B, n, st, mg)
                           : launch_backward_simt<float, 64>(c, q, k, v, dout, dq, dk, dv, dWq, dWk, ph, B, n, st, mg);
    }
    if (res == LINATTN_OK && a && d_a) c->last_launches += 1;
    return res;
}

linattn_status linattn_backward(linattn_ctx* c, const void* q, const void* k, const void* v, const void* dout, void* dq,
                                void* dk, void* dv, float* dWq, float* dWk, int per_head, int B, int H, int n, int d,
                                linattn_dtype dtype, void* stream)
{
    return backward_impl(c, q, k, v, nullptr, 0.f, dout, dq, dk, dv, dWq, dWk, per_head, nullptr, nullptr, B, H, n, d, dtype, stream);
}

linattn_status linattn_backward_mixed(linattn_ctx* c, const void* q, const void* k, const void* v, const void* o_softmax, float r,
                                      const void* dout, void* dq, void* dk, void* dv, float* dWq, float* dWk, int per_head,
                                      void* d_o_softmax, float* dr, int B, int H, int n, int d, linattn_dtype dtype, void* stream)
{
    if (!o_softmax) return LINATTN_ERR_INVALID_ARG;
    return backward_impl(c, q, k, v, o_softmax, r, dout, dq, dk, dv, dWq, dWk, per_head, d_o_softmax, dr, B, H, n, d, dtype, stream);
}

linattn_status linattn_forward_host(linattn_ctx* c, const void* q, const void* k, const void* v, void* out, int B,
                                    int H, int n, int d, linattn_dtype dtype, void* stream)
{
    NvtxRange range("linattn_forward_host");
    linattn_status s = check_forward_args(c, q, k, v, out, B, H, n, d, dtype);
    if (s != LINATTN_OK) return s;
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    const size_t bytes = (size_t)B * H * n * d * elem_size(dtype);
    if (bytes > c->stage_bytes) {
        LA_CUDA(c, cudaStreamSynchronize(st));
        for (void*& p : c->stage) {
            cudaFree(p);
            p = nullptr;
        }
        c->stage_bytes = 0;
        for (void*& p : c->stage) LA_CUDA(c, cudaMalloc(&p, bytes));
        c->stage_bytes = bytes;
    }
    if (!c->copy_in) {
        LA_CUDA(c, cudaStreamCreateWithFlags(&c->copy_in, cudaStreamNonBlocking));
        LA_CUDA(c, cudaStreamCreateWithFlags(&c->copy_out, cudaStreamNonBlocking));
        LA_CUDA(c, cudaEventCreateWithFlags(&c->ev_in, cudaEventDisableTiming));
        LA_CUDA(c, cudaEventCreateWithFlags(&c->ev_done, cudaEventDisableTiming));
        LA_CUDA(c, cudaEventCreateWithFlags(&c->ev_start, cudaEventDisableTiming));
    }
    char* sq = (char*)c->stage[0];
    char* sk = (char*)c->stage[1];
    char* sv = (char*)c->stage[2];
    char* so = (char*)c->stage[3];
    if (c->opt_layout != 0) {
        // token-major layout: the heads are interleaved in memory, so the whole problem goes in one piece
        LA_CUDA(c, cudaMemcpyAsync(sq, q, bytes, cudaMemcpyHostToDevice, st));
        LA_CUDA(c, cudaMemcpyAsync(sk, k, bytes, cudaMemcpyHostToDevice, st));
        LA_CUDA(c, cudaMemcpyAsync(sv, v, bytes, cudaMemcpyHostToDevice, st));
        s = dispatch_forward(c, sq, sk, sv, so, nullptr, 0.f, B, n, d, dtype, st);
        if (s != LINATTN_OK) return s;
        LA_CUDA(c, cudaMemcpyAsync(out, so, bytes, cudaMemcpyDeviceToHost, st));
        LA_CUDA(c, cudaStreamSynchronize(st));
        return LINATTN_OK;
    }
    // [B][H][n][d]: the (b,h) pairs are independent and each is contiguous, so they go through a three-stage pipeline:
    // copies in on one stream, the forward of one pair on the caller's stream, copies out on a third.  The two copy
    // directions overlap, and the first pair is being computed while the rest is still arriving.
    const size_t gbytes = (size_t)n * d * elem_size(dtype);
    const long long G = (long long)B * H;
    LA_CUDA(c, cudaEventRecord(c->ev_start, st));          // work queued on the caller's stream may still use the staging buffers
    LA_CUDA(c, cudaStreamWaitEvent(c->copy_in, c->ev_start, 0));
    LA_CUDA(c, cudaStreamWaitEvent(c->copy_out, c->ev_start, 0));
    linattn_status res = LINATTN_OK;
    cudaError_t ce = cudaSuccess;
    int launches = 0;
    for (long long g = 0; g < G && res == LINATTN_OK && ce == cudaSuccess; ++g) {
        const size_t off = (size_t)g * gbytes;
        ce = cudaMemcpyAsync(sk + off, (const char*)k + off, gbytes, cudaMemcpyHostToDevice, c->copy_in);
        if (ce == cudaSuccess) ce = cudaMemcpyAsync(sv + off, (const char*)v + off, gbytes, cudaMemcpyHostToDevice, c->copy_in);
        if (ce == cudaSuccess) ce = cudaMemcpyAsync(sq + off, (const char*)q + off, gbytes, cudaMemcpyHostToDevice, c->copy_in);
        if (ce == cudaSuccess) ce = cudaEventRecord(c->ev_in, c->copy_in);
        if (ce == cudaSuccess) ce = cudaStreamWaitEvent(st, c->ev_in, 0);
        if (ce != cudaSuccess) break;
        c->view_H = 1;
        c->view_head0 = (int)(g % H);
        c->view_g0 = g;
        res = dispatch_forward(c, sq + off, sk + off, sv + off, so + off, nullptr, 0.f, 1, n, d, dtype, st);
        launches += c->last_launches;
        c->view_H = 0;
        c->view_head0 = 0;
        c->view_g0 = 0;
        if (res != LINATTN_OK) break;
        ce = cudaEventRecord(c->ev_done, st);
        if (ce == cudaSuccess) ce = cudaStreamWaitEvent(c->copy_out, c->ev_done, 0);
        if (ce == cudaSuccess) ce = cudaMemcpyAsync((char*)out + off, so + off, gbytes, cudaMemcpyDeviceToHost, c->copy_out);
    }
    // drain all three streams whatever happened, so that no copy is left in flight on buffers the caller owns
    const cudaError_t e1 = cudaStreamSynchronize(c->copy_in), e2 = cudaStreamSynchronize(st), e3 = cudaStreamSynchronize(c->copy_out);
    c->last_B = B;
    c->last_launches = launches;
    c->state_key.valid = false;
    if (res != LINATTN_OK) return res;
    if (ce != cudaSuccess) return cuda_fail(c, ce, "pipelined host copy");
    if (e1 != cudaSuccess) return cuda_fail(c, e1, "cudaStreamSynchronize(copy_in)");
    if (e2 != cudaSuccess) return cuda_fail(c, e2, "cudaStreamSynchronize(stream)");
    if (e3 != cudaSuccess) return cuda_fail(c, e3, "cudaStreamSynchronize(copy_out)");
    return LINATTN_OK;
}

linattn_status linattn_read_state(linattn_ctx* c, float* S_host, float* z_host, int B, void* stream)
{
    if (!c || B < 1 || B > c->max_B) return LINATTN_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    const size_t dd = (size_t)c->d * c->d, E = dd + c->d;
    const size_t G = (size_t)B * c->H;
    if (S_host)
        LA_CUDA(c, cudaMemcpy2DAsync(S_host, dd * sizeof(float), c->state, E * sizeof(float), dd * sizeof(float), G,
                                     cudaMemcpyDeviceToHost, st));
    if (z_host)
        LA_CUDA(c, cudaMemcpy2DAsync(z_host, c->d * sizeof(float), c->state + dd, E * sizeof(float),
                                     c->d * sizeof(float), G, cudaMemcpyDeviceToHost, st));
    LA_CUDA(c, cudaStreamSynchronize(st));
    if (S_host && c->state_transposed) {
        // the tensor-core kernels keep S as [c][f]; the documented layout is [f][c]
        const int d = c->d;
        for (size_t g = 0; g < G; ++g) {
            float* m = S_host + g * dd;
            for (int i = 0; i < d; ++i)
                for (int j = i + 1; j < d; ++j) {
                    const float t = m[(size_t)i * d + j];
                    m[(size_t)i * d + j] = m[(size_t)j * d + i];
                    m[(size_t)j * d + i] = t;
                }
        }
    }
    return LINATTN_OK;
}

linattn_status linattn_set_option(linattn_ctx* c, linattn_option opt, long long value)
{
    if (!c) return LINATTN_ERR_INVALID_ARG;
    switch (opt) {
        case LINATTN_OPT_SPLITS:
            if (value < 0 || value > kMaxSplits) return LINATTN_ERR_INVALID_ARG;
            c->opt_splits = (int)value;
            return LINATTN_OK;
        case LINATTN_OPT_PATH:
            if (value < 0 || value > 2) return LINATTN_ERR_INVALID_ARG;
            c->opt_path = (int)value;
            return LINATTN_OK;
        case LINATTN_OPT_LAYOUT:
            if (value != 0 && value != 1) return LINATTN_ERR_INVALID_ARG;
            c->opt_layout = (int)value;
            return LINATTN_OK;
        case LINATTN_OPT_KERNEL_FUNCTION:
            if (value != 0 && value != 1) return LINATTN_ERR_INVALID_ARG;
            c->opt_phi = (int)value;
            return LINATTN_OK;
        case LINATTN_OPT_REUSE_STATE:
            if (value != 0 && value != 1) return LINATTN_ERR_INVALID_ARG;
            c->opt_reuse = (int)value;
            return LINATTN_OK;
        case LINATTN_OPT_WAIT_LIMIT_US:
            if (value < 1 || value > 60LL * 1000 * 1000) return LINATTN_ERR_INVALID_ARG;
            c->opt_wait_limit_us = value;
            return LINATTN_OK;
        case LINATTN_OPT_TEST_UNMET_ARRIVAL:
            if (value < 0 || value > 3) return LINATTN_ERR_INVALID_ARG;
            c->opt_unmet = (int)value;
            return LINATTN_OK;
        case LINATTN_OPT_FUSE:
            if (value != 0 && value != 1) return LINATTN_ERR_INVALID_ARG;
            c->opt_fuse = (int)value;
            return LINATTN_OK;
        case LINATTN_OPT_PROFILE: {
            if (value != 0 && value != 1) return LINATTN_ERR_INVALID_ARG;
            DeviceGuard guard(c->device);
            if (value == 1) {
                for (cudaEvent_t& ev : c->prof_ev)
                    if (!ev) LA_CUDA(c, cudaEventCreate(&ev));
                if (!c->profile) {  // a fresh measurement
                    for (int i = 0; i < linattn_ctx::kMaxKernels; ++i) {
                        c->prof_ms[i] = 0.0;
                        c->prof_cnt[i] = 0;
                    }
                }
            } else {
                prof_flush(c);
            }
            c->profile = (value == 1);
            return LINATTN_OK;
        }
    }
    return LINATTN_ERR_INVALID_ARG;
}

linattn_status linattn_check(linattn_ctx* c, void* stream)
{
    if (!c) return LINATTN_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    cudaStream_t st = (cudaStream_t)stream;
    LA_CUDA(c, cudaStreamSynchronize(st));
    unsigned int w = 0;
    LA_CUDA(c, cudaMemcpyAsync(&w, c->err_word, sizeof(w), cudaMemcpyDeviceToHost, st));
    LA_CUDA(c, cudaStreamSynchronize(st));
    if (w != 0) {
        LA_CUDA(c, cudaMemsetAsync(c->err_word, 0, sizeof(w), st));
        LA_CUDA(c, cudaMemsetAsync(c->sync_words, 0, c->sync_bytes, st));  // an aborted launch does not clear its meeting-point counters
        if (w & tc::kErrSmem) snprintf(c->err_text, sizeof(c->err_text), "a kernel's shared-memory window did not hold its layout (code 0x%x)", w);
        else snprintf(c->err_text, sizeof(c->err_text), "device-side wait gave up (code 0x%x)", w);
        return LINATTN_ERR_TIMEOUT;
    }
    return LINATTN_OK;
}

int linattn_profile_get(linattn_ctx* c, int index, const char** name, double* mean_ms, long long* launches,
                        double* algorithmic_bytes)
{
    if (!c || index < 0) return 0;
    {
        DeviceGuard guard(c->device);
        prof_flush(c);
    }
    if (index >= c->prof_n || c->prof_cnt[index] == 0) return 0;
    if (name) *name = c->prof_name[index];
    if (mean_ms) *mean_ms = c->prof_ms[index] / (double)c->prof_cnt[index];
    if (launches) *launches = c->prof_cnt[index];
    if (algorithmic_bytes) *algorithmic_bytes = c->prof_bytes[index];
    return 1;
}

#ifdef LINATTN_TRACE
// Tuning builds only: device buffer that receives the kernels' per-tile timestamps (NULL = off).
linattn_status linattn_set_trace(linattn_ctx* c, long long* device_buffer)
{
    if (!c) return LINATTN_ERR_INVALID_ARG;
    c->trace = device_buffer;
    return LINATTN_OK;
}
#endif

int linattn_last_launch_count(const linattn_ctx* c) { return c ? c->last_launches : 0; }

const char* linattn_last_error(const linattn_ctx* c) { return c ? c->err_text : ""; }

}  // extern "C"
