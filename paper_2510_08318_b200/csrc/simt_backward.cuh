// CUDA-core (fp32 FMA) kernels for the gradients of linear attention with the Hedgehog feature map:
// what the training objective (Eq. 14) back-propagates through each layer that uses Eq. 5 with the phi of Eq. 6.
//
// With dO the gradient that arrives at the layer's output, S = sum_j phi(k_j)^T v_j, z = sum_j phi(k_j),
// den_i = phi(q_i) . z and o_i = phi(q_i) S / den_i, the chain rule gives
//     dnum_i = dO_i / den_i                  dden_i = -(dO_i . o_i) / den_i
//     dphi(q_i) = S dnum_i + dden_i z        dS = sum_i phi(q_i)^T dnum_i       dz = sum_i dden_i phi(q_i)
//     dphi(k_j) = dS v_j + dz                dv_j = dS^T phi(k_j)
// and through phi (p+ = softmax(u), p- = softmax(-u), u = x W)
//     du = p+ (.) (dphi+ - p+ . dphi+) - p- (.) (dphi- - p- . dphi-)       dx = du W^T       dW += x^T du.
//
// Launches of one backward (S and z come from the forward's key-side kernels):
//   qside_bwd     : per (b,h) and per block of token chunks: dq, and the block's partial sums of dS, dz, dW_q
//   combine_state : fixed-order sum of the dS, dz partials (shared with the forward)
//   kside_bwd     : dk, dv and the block's partial sum of dW_k
//   combine_wgrad : fixed-order sum of the weight-gradient partials over blocks, batch and (shared map) heads
// All arithmetic is fp32; every sum has a fixed order, so the gradients are bit-reproducible.
#pragma once
#include "simt_kernels.cuh"

namespace linattn {

template <int D> struct BwdShape {
    static constexpr int M = D / 2;
    static constexpr int P = D + 4;    // pitch of token-major tiles and of the state matrix in shared memory
    static constexpr int PM = M + 4;   // pitch of the du tile
    static constexpr int CG = D / 32;  // float4 column groups per thread in row-times-matrix products
    static constexpr int WA = D / 16;  // rows (input features) of dW per thread
    static constexpr int WB = M / 16;  // columns (logits) of dW per thread
    static constexpr int FB = D / 16, CB = D / 16;  // dS block per thread, as in the forward's key side
};

// Shared-memory floats: W, W^T, state matrix (pitched) + vector, four token tiles, du tile, one scalar per token.
template <int D> constexpr size_t bwd_smem()
{
    return sizeof(float) * (size_t)(2 * D * (D / 2) + D * BwdShape<D>::P + D + 4 * kSimtTokens * BwdShape<D>::P +
                                    kSimtTokens * BwdShape<D>::PM + kSimtTokens);
}

template <int D> struct BwdSmem {
    float *W, *Wt, *A, *a, *x, *y, *phi, *dphi, *du, *dd;
    __device__ explicit BwdSmem(float* base)
    {
        constexpr int M = D / 2, P = BwdShape<D>::P;
        W = base;
        Wt = W + D * M;
        A = Wt + D * M;
        a = A + D * P;
        x = a + D;
        y = x + kSimtTokens * P;
        phi = y + kSimtTokens * P;
        dphi = phi + kSimtTokens * P;
        du = dphi + kSimtTokens * P;
        dd = du + kSimtTokens * BwdShape<D>::PM;
    }
};

// W [D][M] -> W_s as is and Wt_s [M][D];  state [D*D + D] -> A_s [D] rows of pitch P, a_s [D].
template <int D>
__device__ __forceinline__ void bwd_load_constants(const BwdSmem<D>& s, const float* __restrict__ Wg, const float* __restrict__ state)
{
    constexpr int M = D / 2, P = BwdShape<D>::P;
    if (Wg)   // the ReLU kernel function has no weights
        for (int e = threadIdx.x; e < D * M; e += kSimtThreads) {
            const float w = Wg[e];
            s.W[e] = w;
            s.Wt[(e % M) * D + e / M] = w;
        }
    for (int e = threadIdx.x; e < D * D; e += kSimtThreads) s.A[(e / D) * P + e % D] = state[e];
    for (int e = threadIdx.x; e < D; e += kSimtThreads) s.a[e] = state[D * D + e];
}

// res[r][b] = sum_{kk < K} vec[kk] * mat[kk * pitch + r*32 + cg*4 + b]   (one token per 8 threads, cg = lane & 7)
template <int D>
__device__ __forceinline__ void row_times_matrix(const float* __restrict__ vec, int K, const float* __restrict__ mat, int pitch,
                                                 int cg, float (&res)[BwdShape<D>::CG][4])
{
    constexpr int CG = BwdShape<D>::CG;
#pragma unroll
    for (int r = 0; r < CG; ++r)
#pragma unroll
        for (int b = 0; b < 4; ++b) res[r][b] = 0.f;
#pragma unroll 4
    for (int kk = 0; kk < K; ++kk) {
        const float p = vec[kk];
#pragma unroll
        for (int r = 0; r < CG; ++r) {
            const float4 m = *reinterpret_cast<const float4*>(&mat[kk * pitch + r * 32 + cg * 4]);
            res[r][0] = fmaf(p, m.x, res[r][0]);
            res[r][1] = fmaf(p, m.y, res[r][1]);
            res[r][2] = fmaf(p, m.z, res[r][2]);
            res[r][3] = fmaf(p, m.w, res[r][3]);
        }
    }
}

// dphi[t][f] = sum_c A[f][c] * y[t][c] + w_t * a[f],  w_t = dd[t] (scale != nullptr) or 1.
// Thread (tt, jl) covers f = jl + 8r; rows f, f+1, .. of A sit 4 banks apart (pitch D + 4), so the eight lanes of a
// token read their float4s without bank conflicts and the four tokens of a warp share them.
template <int D>
__device__ __forceinline__ void dphi_chunk(const BwdSmem<D>& s, const float* __restrict__ scale)
{
    constexpr int P = BwdShape<D>::P;
    const int tt = threadIdx.x >> 3, jl = threadIdx.x & 7;
    const float w = scale ? scale[tt] : 1.f;
    const float* yr = s.y + tt * P;
    for (int r0 = 0; r0 < D / 8; r0 += 4) {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
        for (int c = 0; c < D; c += 4) {
            const float4 yv = *reinterpret_cast<const float4*>(&yr[c]);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float4 av = *reinterpret_cast<const float4*>(&s.A[(jl + 8 * (r0 + i)) * P + c]);
                acc[i] = fmaf(av.x, yv.x, acc[i]);
                acc[i] = fmaf(av.y, yv.y, acc[i]);
                acc[i] = fmaf(av.z, yv.z, acc[i]);
                acc[i] = fmaf(av.w, yv.w, acc[i]);
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int f = jl + 8 * (r0 + i);
            s.dphi[tt * P + f] = fmaf(w, s.a[f], acc[i]);
        }
    }
}

// Softmax backward of Eq. 6 for the chunk: du[t][j] from phi[t][:] and dphi[t][:].
template <int D>
__device__ __forceinline__ void du_chunk(const BwdSmem<D>& s)
{
    constexpr int M = D / 2, P = BwdShape<D>::P, PM = BwdShape<D>::PM, R = M / 8;
    const int tt = threadIdx.x >> 3, jl = threadIdx.x & 7;
    float pp[R], pn[R], gp[R], gn[R], dotp = 0.f, dotn = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int j = jl + 8 * r;
        pp[r] = s.phi[tt * P + j];
        pn[r] = s.phi[tt * P + M + j];
        gp[r] = s.dphi[tt * P + j];
        gn[r] = s.dphi[tt * P + M + j];
        dotp = fmaf(pp[r], gp[r], dotp);
        dotn = fmaf(pn[r], gn[r], dotn);
    }
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) {
        dotp += __shfl_xor_sync(0xffffffffu, dotp, o);
        dotn += __shfl_xor_sync(0xffffffffu, dotn, o);
    }
#pragma unroll
    for (int r = 0; r < R; ++r) s.du[tt * PM + jl + 8 * r] = pp[r] * (gp[r] - dotp) - pn[r] * (gn[r] - dotn);
}

// dW[c][j] += sum_t x[t][c] * du[t][j] for the chunk; thread (cy, jx) owns c in [cy*WA, +WA), j in [jx*WB, +WB).
// Rows past the valid ones have du = 0.
template <int D>
__device__ __forceinline__ void dw_accumulate(const BwdSmem<D>& s, float (&dw)[BwdShape<D>::WA][BwdShape<D>::WB])
{
    constexpr int P = BwdShape<D>::P, PM = BwdShape<D>::PM, WA = BwdShape<D>::WA, WB = BwdShape<D>::WB;
    const int cy = threadIdx.x >> 4, jx = threadIdx.x & 15;
#pragma unroll 2
    for (int t = 0; t < kSimtTokens; ++t) {
        float xv[WA], dv[WB];
#pragma unroll
        for (int a = 0; a < WA; a += 4) *reinterpret_cast<float4*>(&xv[a]) = *reinterpret_cast<const float4*>(&s.x[t * P + cy * WA + a]);
#pragma unroll
        for (int b = 0; b < WB; b += 2) *reinterpret_cast<float2*>(&dv[b]) = *reinterpret_cast<const float2*>(&s.du[t * PM + jx * WB + b]);
#pragma unroll
        for (int a = 0; a < WA; ++a)
#pragma unroll
            for (int b = 0; b < WB; ++b) dw[a][b] = fmaf(xv[a], dv[b], dw[a][b]);
    }
}

template <int D>
__device__ __forceinline__ void dw_store(float* __restrict__ out, const float (&dw)[BwdShape<D>::WA][BwdShape<D>::WB])
{
    constexpr int M = D / 2, WA = BwdShape<D>::WA, WB = BwdShape<D>::WB;
    const int cy = threadIdx.x >> 4, jx = threadIdx.x & 15;
#pragma unroll
    for (int a = 0; a < WA; ++a)
#pragma unroll
        for (int b = 0; b < WB; ++b) out[(cy * WA + a) * M + jx * WB + b] = dw[a][b];
}

// dx[t][:] = du[t][:] W^T for the chunk's valid tokens, stored in the activations' type.
template <typename T, int D>
__device__ __forceinline__ void dx_store(const BwdSmem<D>& s, T* __restrict__ dst, long long row_stride, int valid)
{
    constexpr int M = D / 2, PM = BwdShape<D>::PM, CG = BwdShape<D>::CG;
    const int tt = threadIdx.x >> 3, cg = threadIdx.x & 7;
    float dx[CG][4];
    row_times_matrix<D>(s.du + tt * PM, M, s.Wt, D, cg, dx);
    if (tt < valid) {
#pragma unroll
        for (int r = 0; r < CG; ++r)
#pragma unroll
            for (int b = 0; b < 4; ++b) store_out(&dst[(size_t)tt * row_stride + r * 32 + cg * 4 + b], dx[r][b]);
    }
}

// ReLU kernel function, phi(x) = max(x, 0): dx[t][c] = dphi[t][c] where x[t][c] > 0, else 0 (no weights, no softmax).
template <typename T, int D>
__device__ __forceinline__ void relu_dx_store(const BwdSmem<D>& s, T* __restrict__ dst, long long row_stride, int valid)
{
    constexpr int P = BwdShape<D>::P;
    for (int e = threadIdx.x; e < kSimtTokens * D; e += kSimtThreads) {
        const int r = e / D, c = e % D;
        if (r < valid) store_out(&dst[(size_t)r * row_stride + c], s.x[r * P + c] > 0.f ? s.dphi[r * P + c] : 0.f);
    }
}

// Sum of one value per thread over the block in a fixed order (thread 0 adds them up); every thread gets the result.
__device__ __forceinline__ float block_sum_ordered(float v, float* scratch)
{
    __syncthreads();
    scratch[threadIdx.x] = v;
    __syncthreads();
    float acc = 0.f;
    if (threadIdx.x == 0) {
        for (int i = 0; i < kSimtThreads; ++i) acc += scratch[i];
        scratch[0] = acc;
    }
    __syncthreads();
    return scratch[0];
}

// grid = (blocks_per_group, G).  Block x handles chunks x, x + gridDim.x, ... of kSimtTokens tokens.
//   relu      : 1 = the ReLU kernel function instead of Eq. 6 (no weights: Wq is NULL, part_w is not written)
//   mix_a, lin_scale, part_dr : Eq. 8.  The gradient that reaches the linear branch is lin_scale * dout (lin_scale = 1 - r^);
//               when mix_a (the softmax branch's output, laid out like q) is given, part_dr [G][gridDim.x] receives the
//               block's sum of dout . (a - o), the terms of dL/dr
//   state     : [G][D*D + D]  S row-major [f][c], then z   (from the forward's key side)
//   dq        : same layout and type as q
//   part_state: [G][gridDim.x][D*D + D]  the block's sums of dS ([f][c]) and dz
//   part_w    : [G][gridDim.x][D*M]      the block's sum of dW_q
template <typename T, int D>
__global__ void __launch_bounds__(kSimtThreads)
qside_bwd(const T* __restrict__ q, const T* __restrict__ dout, const float* __restrict__ Wq, const float* __restrict__ state,
          T* __restrict__ dq, float* __restrict__ part_state, float* __restrict__ part_w, int H, int n, ActStrides st, int relu,
          const T* __restrict__ mix_a, float lin_scale, float* __restrict__ part_dr)
{
    using Sh = BwdShape<D>;
    constexpr int M = Sh::M, P = Sh::P, CG = Sh::CG, FB = Sh::FB, CB = Sh::CB;
    extern __shared__ __align__(16) float smem[];
    const BwdSmem<D> s(smem);
    const int g = blockIdx.y, tid = threadIdx.x;
    bwd_load_constants<D>(s, relu ? nullptr : Wq + (size_t)(g % H) * D * M, state + (size_t)g * (D * D + D));

    const T* qg = q + st.base(g, H);
    const T* gg = dout + st.base(g, H);
    const T* ag = mix_a ? mix_a + st.base(g, H) : nullptr;
    float dr_acc = 0.f;   // this thread's share of sum dout . (a - o)
    T* dqg = dq + st.base(g, H);
    const int tt = tid >> 3, cg = tid & 7;
    const int fy = tid >> 4, cx = tid & 15;
    const int nchunks = (n + kSimtTokens - 1) / kSimtTokens;

    float dS[FB][CB], dz[FB], dw[Sh::WA][Sh::WB];
#pragma unroll
    for (int a = 0; a < FB; ++a) {
        dz[a] = 0.f;
#pragma unroll
        for (int b = 0; b < CB; ++b) dS[a][b] = 0.f;
    }
#pragma unroll
    for (int a = 0; a < Sh::WA; ++a)
#pragma unroll
        for (int b = 0; b < Sh::WB; ++b) dw[a][b] = 0.f;

    for (int ch = blockIdx.x; ch < nchunks; ch += gridDim.x) {
        const int t = ch * kSimtTokens;
        const int valid = min(kSimtTokens, n - t);
        __syncthreads();
        load_chunk<T, D>(qg + (size_t)t * st.token, st.token, s.x, valid);
        load_chunk<T, D>(gg + (size_t)t * st.token, st.token, s.y, valid);
        __syncthreads();
        if (relu) relu_chunk<D>(s.x, s.phi, valid);
        else feature_map_chunk<D>(s.x, s.W, s.phi, valid);   // rows past `valid` get phi = 0
        __syncthreads();
        {
            // forward quantities of the token, then dnum (over dO in place) and dden
            float num[CG][4];
            row_times_matrix<D>(s.phi + tt * P, D, s.A, P, cg, num);
            float den = 0.f;
#pragma unroll 8
            for (int f = 0; f < D; ++f) den = fmaf(s.phi[tt * P + f], s.a[f], den);
            const float inv = (tt < valid) ? 1.f / den : 0.f;
            const float sc = lin_scale * inv;   // the linear branch's incoming gradient is lin_scale * dO
            float go = 0.f;
#pragma unroll
            for (int r = 0; r < CG; ++r) {
                float4* gp = reinterpret_cast<float4*>(&s.y[tt * P + r * 32 + cg * 4]);
                float4 gv = *gp;
                go = fmaf(gv.x, num[r][0] * inv, go);
                go = fmaf(gv.y, num[r][1] * inv, go);
                go = fmaf(gv.z, num[r][2] * inv, go);
                go = fmaf(gv.w, num[r][3] * inv, go);
                if (ag && tt < valid) {   // Eq. 8: dO . a, the softmax branch's part of dL/dr
                    const T* ap = ag + (size_t)(t + tt) * st.token + r * 32 + cg * 4;
                    dr_acc = fmaf(gv.x, to_f32(ap[0]), dr_acc);
                    dr_acc = fmaf(gv.y, to_f32(ap[1]), dr_acc);
                    dr_acc = fmaf(gv.z, to_f32(ap[2]), dr_acc);
                    dr_acc = fmaf(gv.w, to_f32(ap[3]), dr_acc);
                }
                gv.x *= sc; gv.y *= sc; gv.z *= sc; gv.w *= sc;
                *gp = gv;
            }
            dr_acc -= go;   // ... minus dO . o, each thread its own columns' share
#pragma unroll
            for (int o = 1; o < 8; o <<= 1) go += __shfl_xor_sync(0xffffffffu, go, o);
            if (cg == 0) s.dd[tt] = -go * sc;
        }
        __syncthreads();
        dphi_chunk<D>(s, s.dd);
        // dS += phi^T dnum, dz += phi^T dden
#pragma unroll 2
        for (int r = 0; r < kSimtTokens; ++r) {
            float ph[FB], gv[CB];
            const float ddr = s.dd[r];
#pragma unroll
            for (int a = 0; a < FB; a += 4)
                *reinterpret_cast<float4*>(&ph[a]) = *reinterpret_cast<const float4*>(&s.phi[r * P + fy * FB + a]);
#pragma unroll
            for (int b = 0; b < CB; b += 4)
                *reinterpret_cast<float4*>(&gv[b]) = *reinterpret_cast<const float4*>(&s.y[r * P + (b / 4) * 64 + cx * 4]);
#pragma unroll
            for (int a = 0; a < FB; ++a) {
                dz[a] = fmaf(ph[a], ddr, dz[a]);
#pragma unroll
                for (int b = 0; b < CB; ++b) dS[a][b] = fmaf(ph[a], gv[b], dS[a][b]);
            }
        }
        __syncthreads();
        if (relu) {
            relu_dx_store<T, D>(s, dqg + (size_t)t * st.token, st.token, valid);
        } else {
            du_chunk<D>(s);
            __syncthreads();
            dx_store<T, D>(s, dqg + (size_t)t * st.token, st.token, valid);
            dw_accumulate<D>(s, dw);
        }
    }

    const size_t slot = (size_t)g * gridDim.x + blockIdx.x;
    if (part_dr) {
        const float total = block_sum_ordered(dr_acc, s.phi);   // the token tiles are free now
        if (tid == 0) part_dr[slot] = total;
    }
    float* ps = part_state + slot * (D * D + D);
#pragma unroll
    for (int a = 0; a < FB; ++a) {
        const int f = fy * FB + a;
#pragma unroll
        for (int b = 0; b < CB; b += 4)
            *reinterpret_cast<float4*>(&ps[f * D + (b / 4) * 64 + cx * 4]) = *reinterpret_cast<float4*>(&dS[a][b]);
        if (cx == 0) ps[D * D + f] = dz[a];
    }
    if (!relu) dw_store<D>(part_w + slot * (D * M), dw);
}

// grid = (blocks_per_group, G).
//   dstate: [G][D*D + D]  dS row-major [f][c], then dz
//   dk, dv: same layout and type as k, v
//   part_w: [G][gridDim.x][D*M]  the block's sum of dW_k
template <typename T, int D>
__global__ void __launch_bounds__(kSimtThreads)
kside_bwd(const T* __restrict__ k, const T* __restrict__ v, const float* __restrict__ Wk, const float* __restrict__ dstate,
          T* __restrict__ dk, T* __restrict__ dv, float* __restrict__ part_w, int H, int n, ActStrides st, int relu)
{
    using Sh = BwdShape<D>;
    constexpr int M = Sh::M, P = Sh::P, CG = Sh::CG;
    extern __shared__ __align__(16) float smem[];
    const BwdSmem<D> s(smem);
    const int g = blockIdx.y, tid = threadIdx.x;
    bwd_load_constants<D>(s, relu ? nullptr : Wk + (size_t)(g % H) * D * M, dstate + (size_t)g * (D * D + D));

    const T* kg = k + st.base(g, H);
    const T* vg = v + st.base(g, H);
    T* dkg = dk + st.base(g, H);
    T* dvg = dv + st.base(g, H);
    const int tt = tid >> 3, cg = tid & 7;
    const int nchunks = (n + kSimtTokens - 1) / kSimtTokens;

    float dw[Sh::WA][Sh::WB];
#pragma unroll
    for (int a = 0; a < Sh::WA; ++a)
#pragma unroll
        for (int b = 0; b < Sh::WB; ++b) dw[a][b] = 0.f;

    for (int ch = blockIdx.x; ch < nchunks; ch += gridDim.x) {
        const int t = ch * kSimtTokens;
        const int valid = min(kSimtTokens, n - t);
        __syncthreads();
        load_chunk<T, D>(kg + (size_t)t * st.token, st.token, s.x, valid);
        load_chunk<T, D>(vg + (size_t)t * st.token, st.token, s.y, valid);
        __syncthreads();
        if (relu) relu_chunk<D>(s.x, s.phi, valid);
        else feature_map_chunk<D>(s.x, s.W, s.phi, valid);
        __syncthreads();
        dphi_chunk<D>(s, nullptr);
        {
            float r_dv[CG][4];
            row_times_matrix<D>(s.phi + tt * P, D, s.A, P, cg, r_dv);
            if (tt < valid) {
#pragma unroll
                for (int r = 0; r < CG; ++r)
#pragma unroll
                    for (int b = 0; b < 4; ++b)
                        store_out(&dvg[(size_t)(t + tt) * st.token + r * 32 + cg * 4 + b], r_dv[r][b]);
            }
        }
        __syncthreads();
        if (relu) {
            relu_dx_store<T, D>(s, dkg + (size_t)t * st.token, st.token, valid);
        } else {
            du_chunk<D>(s);
            __syncthreads();
            dx_store<T, D>(s, dkg + (size_t)t * st.token, st.token, valid);
            dw_accumulate<D>(s, dw);
        }
    }
    if (!relu) dw_store<D>(part_w + ((size_t)g * gridDim.x + blockIdx.x) * (D * M), dw);
}

// dW[w][e] = sum over the groups g that use weight matrix w (per_head: g % H == w; shared: all g), g ascending, and
// over that group's blocks, ascending.  grid = (ceil(DM/256), per_head ? H : 1).
static __global__ void __launch_bounds__(256)
combine_wgrad(const float* __restrict__ part_w, float* __restrict__ dW, int blocks, int G, int H, int DM, int per_head)
{
    const int e = blockIdx.x * 256 + threadIdx.x;
    if (e >= DM) return;
    const int w = blockIdx.y;
    float acc = 0.f;
    for (int g = per_head ? w : 0; g < G; g += per_head ? H : 1) {
        const float* p = part_w + (size_t)g * blocks * DM + e;
        for (int b = 0; b < blocks; ++b) acc += p[(size_t)b * DM];
    }
    dW[(size_t)w * DM + e] = acc;
}

// Eq. 8: dL/dr = sum of the partial sums of dout . (a - o), in index order, if r lies in [0, 1] (the clip passes the
// gradient on the closed interval), else 0.  One thread.
static __global__ void combine_dr(const float* __restrict__ part_dr, int count, int in_range, float* __restrict__ dr)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    float acc = 0.f;
    for (int i = 0; i < count; ++i) acc += part_dr[i];
    *dr = in_range ? acc : 0.f;
}

// Eq. 8: the gradient that reaches the softmax branch, d_a = r^ * dout, element by element (any layout: `count` elements).
template <typename T>
static __global__ void __launch_bounds__(256) scale_copy(const T* __restrict__ src, T* __restrict__ dst, size_t count, float f)
{
    for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < count; i += (size_t)gridDim.x * 256) store_out(&dst[i], f * to_f32(src[i]));
}

}  // namespace linattn
