// linattn_forward_noalloc: the CUDA-core forward with its scratch memory in a fixed device array.
//
// Some callers cannot allocate device memory when they call into this library: code running
// inside a memory pool it does not own, a host thread of a serving loop where cudaMalloc's
// implicit device synchronisation would stall every other stream, or a plug-in that has been
// handed pointers and a stream and nothing else.  For them this file keeps the key-side
// partial sums and the combined S, z (Eq. 5) in a file-scope __device__ array of fixed size,
// so the entry point needs no context and calls no allocator at all.
#include "linattn.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "simt_kernels.cuh"

using namespace linattn;

namespace {

// Limits of the fixed scratch (stated in include/linattn.h).
constexpr int kNoAllocMaxGroups = 16;        // B*H
constexpr int kNoAllocPartialSlots = 64;     // (b,h) pairs x splits
constexpr int kNoAllocMaxE = 128 * 128 + 128;  // floats per slot at d = 128
constexpr size_t kScratchFloats = (size_t)(kNoAllocPartialSlots + kNoAllocMaxGroups) * kNoAllocMaxE;

// Every GPU that loads the library holds these ~5.3 MB until the process exits.
static __device__ __align__(256) float g_noalloc_scratch[kScratchFloats];

// Host-side caches, filled by the first call on each device.  They are plain variables: two host threads that make
// their FIRST call on a device at the same moment would both run the set-up (each stores the same values), so the
// documented rule is to make the first call on a device from one thread.
constexpr int kMaxDevices = 64;
float* g_scratch_ptr[kMaxDevices] = {};  // device address of g_noalloc_scratch on each device, set up on first use
bool g_attr_done[kMaxDevices][4] = {};
int g_cc_major[kMaxDevices] = {};        // compute capability (major) of each device, 0 = not asked yet

// The array's name is only a host-side handle here; kernels need its device address, which the
// runtime gives per device.  Done once per device, with that device current.
linattn_status scratch_for_current_device(int dev, float** out)
{
    if (dev < 0 || dev >= kMaxDevices) return LINATTN_ERR_UNSUPPORTED;
    if (g_cc_major[dev] == 0) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
            cudaGetLastError();
            return LINATTN_ERR_CUDA;
        }
        g_cc_major[dev] = major;
    }
    if (g_cc_major[dev] != 10) return LINATTN_ERR_UNSUPPORTED;   // the library is built for sm_100a only
    if (!g_scratch_ptr[dev]) {
        float* p = nullptr;
        if (cudaGetSymbolAddress((void**)&p, g_noalloc_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return LINATTN_ERR_CUDA;
        }
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return LINATTN_OK;
}

template <typename T, int D>
linattn_status run(int dev, int slot, float* scratch, const T* q, const T* k, const T* v, T* out, const float* Wq,
                   const float* Wk, int Hw, long long G, int n, cudaStream_t st)
{
    constexpr int E = D * D + D;
    if (!g_attr_done[dev][slot]) {
        if (cudaFuncSetAttribute(kside_simt<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kside_simt_smem<D>()) != cudaSuccess ||
            cudaFuncSetAttribute(qside_simt<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)qside_simt_smem<D>()) != cudaSuccess) {
            cudaGetLastError();
            return LINATTN_ERR_CUDA;
        }
        g_attr_done[dev][slot] = true;
    }
    // as many splits of the token range as the fixed partial area holds, at least 256 tokens each
    long long splits = kNoAllocPartialSlots / G;
    const long long by_len = ((long long)n + 255) / 256;
    if (splits > by_len) splits = by_len;
    if (splits < 1) splits = 1;
    int chunk = (int)((n + splits - 1) / splits);
    chunk = (chunk + kSimtTokens - 1) / kSimtTokens * kSimtTokens;
    splits = (n + chunk - 1) / chunk;

    float* partial = scratch;                                              // [G*splits][E], fully overwritten
    float* state = scratch + (size_t)kNoAllocPartialSlots * kNoAllocMaxE;  // [G][E], fully overwritten
    kside_simt<T, D><<<dim3((unsigned)splits, (unsigned)G), kSimtThreads, kside_simt_smem<D>(), st>>>(
        k, v, Wk, partial, Hw, n, chunk, ActStrides{D, (long long)n * D, (long long)Hw * n * D}, 0);
    combine_state<<<dim3((E + 255) / 256, (unsigned)G), 256, 0, st>>>(partial, state, (int)splits, E);
    const int nchunks = (n + kSimtTokens - 1) / kSimtTokens;
    long long per_group = (2LL * 148 + G - 1) / G;
    if (per_group > nchunks) per_group = nchunks;
    qside_simt<T, D><<<dim3((unsigned)per_group, (unsigned)G), kSimtThreads, qside_simt_smem<D>(), st>>>(
        q, Wq, state, out, Hw, n, (const T*)nullptr, 0.f, ActStrides{D, (long long)n * D, (long long)Hw * n * D}, 0);
    if (cudaGetLastError() != cudaSuccess) return LINATTN_ERR_CUDA;
    return LINATTN_OK;
}

}  // namespace

extern "C" linattn_status linattn_forward_noalloc(const void* q, const void* k, const void* v, void* out,
                                                  const float* Wq, const float* Wk, int per_head, int B, int H, int n,
                                                  int d, linattn_dtype dtype, void* stream)
{
    if (!q || !k || !v || !out || !Wq || !Wk) return LINATTN_ERR_INVALID_ARG;
    if (dtype != LINATTN_F32 && dtype != LINATTN_BF16) return LINATTN_ERR_UNSUPPORTED;
    if (d != 64 && d != 128) return LINATTN_ERR_UNSUPPORTED;
    if (B < 1 || H < 1 || n < 1) return LINATTN_ERR_INVALID_ARG;
    const long long G = (long long)B * H;
    if (G > kNoAllocMaxGroups) return LINATTN_ERR_WORKSPACE;  // beyond the fixed scratch
    const uintptr_t bits = (uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out | (uintptr_t)Wq | (uintptr_t)Wk;
    if (bits & 15u) return LINATTN_ERR_INVALID_ARG;
    // out is written while q, k, v are still being read: it must not overlap any of them
    const size_t bytes = (size_t)G * (size_t)n * (size_t)d * (dtype == LINATTN_BF16 ? 2u : 4u);
    const uintptr_t o0 = (uintptr_t)out;
    for (const void* in : {q, k, v}) {
        const uintptr_t i0 = (uintptr_t)in;
        if (o0 < i0 + bytes && i0 < o0 + bytes) return LINATTN_ERR_INVALID_ARG;
    }

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return LINATTN_ERR_CUDA;
    }
    float* scratch = nullptr;
    linattn_status s = scratch_for_current_device(dev, &scratch);
    if (s != LINATTN_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    const int Hw = per_head ? H : 1;  // the kernels pick weight matrix (b*H + h) % Hw
    if (dtype == LINATTN_BF16) {
        using T = __nv_bfloat16;
        return d == 128 ? run<T, 128>(dev, 0, scratch, (const T*)q, (const T*)k, (const T*)v, (T*)out, Wq, Wk, Hw, G, n, st)
                        : run<T, 64>(dev, 1, scratch, (const T*)q, (const T*)k, (const T*)v, (T*)out, Wq, Wk, Hw, G, n, st);
    }
    return d == 128 ? run<float, 128>(dev, 2, scratch, (const float*)q, (const float*)k, (const float*)v, (float*)out, Wq, Wk, Hw, G, n, st)
                    : run<float, 64>(dev, 3, scratch, (const float*)q, (const float*)k, (const float*)v, (float*)out, Wq, Wk, Hw, G, n, st);
}
