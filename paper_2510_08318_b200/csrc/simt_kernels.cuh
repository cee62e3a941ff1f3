// CUDA-core (fp32 FMA) kernels for linear attention with the Hedgehog feature map.
//
// These are the general path: fp32 and bf16 storage, d = 64 or 128, any n >= 1.  All arithmetic
// is fp32.  Three launches per forward:
//   kside_simt   : per (b,h) and per split of the token range, phi(k) (Eq. 6) and the partial
//                  sums of S = sum_j phi(k_j)^T v_j and z = sum_j phi(k_j) (Eq. 5)
//   combine_state: fixed-order sum of the partials (deterministic)
//   qside_simt   : phi(q) (Eq. 6), o_i = phi(q_i) S / (phi(q_i) . z) (Eq. 5)
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace linattn {

constexpr int kSimtThreads = 256;
constexpr int kSimtTokens = 32;  // tokens per chunk in both SIMT kernels

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void store_out(float* p, float x) { *p = x; }
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

// Row pitch (floats) of token-major shared tiles: +4 keeps 16-byte alignment and moves
// consecutive rows to different banks.
template <int D> struct SimtShape {
    static constexpr int M = D / 2;
    static constexpr int PITCH = D + 4;
};

// Eq. 6 for kSimtTokens rows held in x_s (fp32, pitch PITCH) -> phi_s (pitch PITCH).
// Rows >= valid get phi = 0 so that they add nothing to S, z.  8 threads share one row.
template <int D>
__device__ __forceinline__ void feature_map_chunk(const float* __restrict__ x_s, const float* __restrict__ W_s,
                                                  float* __restrict__ phi_s, int valid)
{
    constexpr int M = SimtShape<D>::M, P = SimtShape<D>::PITCH;
    constexpr int R = M / 8;  // logits per thread
    const int tid = threadIdx.x;
    const int tt = tid >> 3, jl = tid & 7;
    float u[R];
#pragma unroll
    for (int r = 0; r < R; ++r) u[r] = 0.f;
    const float* xr = x_s + tt * P;
#pragma unroll 4
    for (int c = 0; c < D; ++c) {
        const float xv = xr[c];
#pragma unroll
        for (int r = 0; r < R; ++r) u[r] = fmaf(xv, W_s[c * M + jl + 8 * r], u[r]);
    }
    float umax = u[0], umin = u[0];
#pragma unroll
    for (int r = 1; r < R; ++r) { umax = fmaxf(umax, u[r]); umin = fminf(umin, u[r]); }
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) {
        umax = fmaxf(umax, __shfl_xor_sync(0xffffffffu, umax, o));
        umin = fminf(umin, __shfl_xor_sync(0xffffffffu, umin, o));
    }
    float ep[R], en[R], sp = 0.f, sn = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        ep[r] = expf(u[r] - umax);   // softmax(+u), max-subtracted
        en[r] = expf(umin - u[r]);   // softmax(-u): max(-u) = -min(u)
        sp += ep[r];
        sn += en[r];
    }
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) {
        sp += __shfl_xor_sync(0xffffffffu, sp, o);
        sn += __shfl_xor_sync(0xffffffffu, sn, o);
    }
    const float keep = (tt < valid) ? 1.f : 0.f;
    const float ip = keep / sp, in = keep / sn;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        phi_s[tt * P + jl + 8 * r] = ep[r] * ip;
        phi_s[tt * P + M + jl + 8 * r] = en[r] * in;
    }
}

// The ReLU kernel function, phi(x) = max(x, 0) element by element, for the chunk; rows >= valid get phi = 0.
template <int D>
__device__ __forceinline__ void relu_chunk(const float* __restrict__ x_s, float* __restrict__ phi_s, int valid)
{
    constexpr int P = SimtShape<D>::PITCH;
    for (int e = threadIdx.x; e < kSimtTokens * D; e += kSimtThreads) {
        const int r = e / D, c = e % D;
        phi_s[r * P + c] = (r < valid) ? fmaxf(x_s[r * P + c], 0.f) : 0.f;
    }
}

// Load `rows` x D elements starting at src (row-major, contiguous) into dst (fp32, pitch PITCH);
// rows in [valid, kSimtTokens) are zero-filled.
template <typename T, int D>
__device__ __forceinline__ void load_chunk(const T* __restrict__ src, long long row_stride, float* __restrict__ dst, int valid)
{
    constexpr int P = SimtShape<D>::PITCH;
    for (int e = threadIdx.x; e < kSimtTokens * D; e += kSimtThreads) {
        const int r = e / D, c = e % D;
        dst[r * P + c] = (r < valid) ? to_f32(src[(size_t)r * row_stride + c]) : 0.f;
    }
}

// Element strides of the activations [batch][head][token][feature] (feature contiguous) in memory.
struct ActStrides {
    long long token, head, batch;
    __device__ __forceinline__ size_t base(int g, int H) const { return (size_t)(g / H) * batch + (size_t)(g % H) * head; }
};

template <int D> constexpr size_t kside_simt_smem()
{
    return sizeof(float) * (size_t)(D * (D / 2) + 3 * kSimtTokens * SimtShape<D>::PITCH);
}

// grid = (splits, G).  Split s of group g covers tokens [s*chunk, min(n, (s+1)*chunk)).
// partial: [G][splits][D*D + D] floats (S row-major [f][c], then z).
template <typename T, int D>
__global__ void __launch_bounds__(kSimtThreads)
kside_simt(const T* __restrict__ k, const T* __restrict__ v, const float* __restrict__ Wk /*[H][D][M]*/,
           float* __restrict__ partial, int H, int n, int chunk, ActStrides st, int relu)
{
    constexpr int M = SimtShape<D>::M, P = SimtShape<D>::PITCH;
    constexpr int FB = D / 16;           // f rows per thread (8 or 4)
    constexpr int CB = D / 16;           // c columns per thread (8 or 4), as CB/4 float4 groups
    extern __shared__ __align__(16) float smem[];
    float* W_s = smem;
    float* k_s = W_s + D * M;
    float* v_s = k_s + kSimtTokens * P;
    float* phi_s = v_s + kSimtTokens * P;

    const int g = blockIdx.y, s = blockIdx.x, splits = gridDim.x;
    const int tid = threadIdx.x;
    const float* Wg = Wk + (size_t)(g % H) * D * M;
    for (int e = tid; e < D * M; e += kSimtThreads) W_s[e] = Wg[e];

    const int t0 = s * chunk, t1 = min(n, t0 + chunk);
    const int fy = tid >> 4, cx = tid & 15;
    float acc[FB][CB];
    float zacc[FB];
#pragma unroll
    for (int a = 0; a < FB; ++a) {
        zacc[a] = 0.f;
#pragma unroll
        for (int b = 0; b < CB; ++b) acc[a][b] = 0.f;
    }
    const T* kg = k + st.base(g, H);
    const T* vg = v + st.base(g, H);

    for (int t = t0; t < t1; t += kSimtTokens) {
        const int valid = min(kSimtTokens, t1 - t);
        __syncthreads();  // previous chunk fully consumed (and W_s visible on the first pass)
        load_chunk<T, D>(kg + (size_t)t * st.token, st.token, k_s, valid);
        load_chunk<T, D>(vg + (size_t)t * st.token, st.token, v_s, valid);
        __syncthreads();
        if (relu) relu_chunk<D>(k_s, phi_s, valid);
        else feature_map_chunk<D>(k_s, W_s, phi_s, valid);
        __syncthreads();
#pragma unroll 2
        for (int r = 0; r < kSimtTokens; ++r) {
            float ph[FB], vv[CB];
#pragma unroll
            for (int a = 0; a < FB; a += 4)
                *reinterpret_cast<float4*>(&ph[a]) = *reinterpret_cast<const float4*>(&phi_s[r * P + fy * FB + a]);
#pragma unroll
            for (int b = 0; b < CB; b += 4)
                *reinterpret_cast<float4*>(&vv[b]) =
                    *reinterpret_cast<const float4*>(&v_s[r * P + (b / 4) * 64 + cx * 4]);
#pragma unroll
            for (int a = 0; a < FB; ++a) {
                zacc[a] += ph[a];
#pragma unroll
                for (int b = 0; b < CB; ++b) acc[a][b] = fmaf(ph[a], vv[b], acc[a][b]);
            }
        }
    }

    float* out = partial + ((size_t)g * splits + s) * (D * D + D);
#pragma unroll
    for (int a = 0; a < FB; ++a) {
        const int f = fy * FB + a;
#pragma unroll
        for (int b = 0; b < CB; b += 4)
            *reinterpret_cast<float4*>(&out[f * D + (b / 4) * 64 + cx * 4]) = *reinterpret_cast<float4*>(&acc[a][b]);
        if (cx == 0) out[D * D + f] = zacc[a];
    }
}

// state[g][e] = sum_{s=0..splits-1} partial[g][s][e], s ascending.  grid = (ceil(E/256), G), E = D*D + D.
static __global__ void __launch_bounds__(256)
combine_state(const float* __restrict__ partial, float* __restrict__ state, int splits, int E)
{
    const int e = blockIdx.x * 256 + threadIdx.x;
    if (e >= E) return;
    const int g = blockIdx.y;
    const float* p = partial + (size_t)g * splits * E + e;
    float acc = 0.f;
    for (int s = 0; s < splits; ++s) acc += p[(size_t)s * E];
    state[(size_t)g * E + e] = acc;
}

template <int D> constexpr size_t qside_simt_smem()
{
    return sizeof(float) * (size_t)(D * (D / 2) + D * D + D + 2 * kSimtTokens * SimtShape<D>::PITCH);
}

// grid = (blocks_per_group, G).  Block x handles chunks x, x + gridDim.x, ... of kSimtTokens tokens.
// state: [G][D*D + D] floats (S then z).
// relu != 0: the ReLU kernel function instead of Eq. 6 (Wq / Wk are then loaded but not used).
// mix != nullptr: Eq. 8, out = mix_r * mix + (1 - mix_r) * (Eq. 5), mix = output of the softmax-attention branch
// ([G][n][D], may be the same buffer as out), mix_r already clipped into [0, 1].
template <typename T, int D>
__global__ void __launch_bounds__(kSimtThreads)
qside_simt(const T* __restrict__ q, const float* __restrict__ Wq, const float* __restrict__ state,
           T* out, int H, int n, const T* mix, float mix_r, ActStrides st, int relu)
{
    constexpr int M = SimtShape<D>::M, P = SimtShape<D>::PITCH;
    constexpr int CG = D / 32;  // float4 column groups per thread (4 or 2)
    extern __shared__ __align__(16) float smem[];
    float* W_s = smem;
    float* S_s = W_s + D * M;
    float* z_s = S_s + D * D;
    float* q_s = z_s + D;
    float* phi_s = q_s + kSimtTokens * P;

    const int g = blockIdx.y, tid = threadIdx.x;
    const float* Wg = Wq + (size_t)(g % H) * D * M;
    const float* Sg = state + (size_t)g * (D * D + D);
    for (int e = tid; e < D * M; e += kSimtThreads) W_s[e] = Wg[e];
    for (int e = tid; e < D * D + D; e += kSimtThreads) S_s[e] = Sg[e];  // z_s follows S_s

    const T* qg = q + st.base(g, H);
    T* og = out + st.base(g, H);
    const int tt = tid >> 3, cg = tid & 7;
    const int nchunks = (n + kSimtTokens - 1) / kSimtTokens;

    for (int ch = blockIdx.x; ch < nchunks; ch += gridDim.x) {
        const int t = ch * kSimtTokens;
        const int valid = min(kSimtTokens, n - t);
        __syncthreads();
        load_chunk<T, D>(qg + (size_t)t * st.token, st.token, q_s, valid);
        __syncthreads();
        // tail rows see zero-filled q: their phi is finite (Eq. 6) or zero (ReLU); their outputs are never stored
        if (relu) relu_chunk<D>(q_s, phi_s, kSimtTokens);
        else feature_map_chunk<D>(q_s, W_s, phi_s, kSimtTokens);
        __syncthreads();
        float num[CG][4];
#pragma unroll
        for (int r = 0; r < CG; ++r)
#pragma unroll
            for (int b = 0; b < 4; ++b) num[r][b] = 0.f;
        float den = 0.f;
        const float* pr = phi_s + tt * P;
#pragma unroll 4
        for (int f = 0; f < D; ++f) {
            const float p = pr[f];
            den = fmaf(p, z_s[f], den);
#pragma unroll
            for (int r = 0; r < CG; ++r) {
                const float4 sv = *reinterpret_cast<const float4*>(&S_s[f * D + r * 32 + cg * 4]);
                num[r][0] = fmaf(p, sv.x, num[r][0]);
                num[r][1] = fmaf(p, sv.y, num[r][1]);
                num[r][2] = fmaf(p, sv.z, num[r][2]);
                num[r][3] = fmaf(p, sv.w, num[r][3]);
            }
        }
        if (tt < valid) {
            const float inv = 1.f / den;
            const T* mg = mix ? mix + st.base(g, H) : nullptr;
#pragma unroll
            for (int r = 0; r < CG; ++r)
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const size_t e = (size_t)(t + tt) * st.token + r * 32 + cg * 4 + b;
                    const float lin = num[r][b] * inv;
                    store_out(&og[e], mg ? fmaf(lin, 1.f - mix_r, mix_r * to_f32(mg[e])) : lin);
                }
        }
    }
}

// Feature-map weights: any supported storage type -> fp32 [H][D][M]; src is [H][D][M] or, when
// per_head == 0, a single [D][M] replicated to every head.
template <typename T>
__global__ void convert_weights(const T* __restrict__ src, float* __restrict__ dst, int H, int DM, int per_head)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)H * DM) return;
    dst[i] = to_f32(src[per_head ? i : i % DM]);
}

}  // namespace linattn
