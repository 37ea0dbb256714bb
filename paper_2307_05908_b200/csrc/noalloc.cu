// Head + top-k entry point that needs no device allocation from anyone.
//
// Some callers can hand this library input and output buffers but cannot obtain scratch memory at
// the time of the call: code running inside a memory pool that is already fully carved up, a
// plugin invoked while its host application has forbidden cudaMalloc (allocation synchronises
// the whole device and would stall the other streams of a serving process), or a process whose
// memory budget was fixed at start-up.  For them the merge scratch of the head kernel lives in a
// file-scope device array that is part of the loaded library image.
#include <cuda_runtime.h>

#include "../../include/ppd.h"
#include "common.cuh"
#include "gemv.cuh"

using namespace ppd;

namespace {

// per-CTA candidate lists + arrival ticket, then the merged top-8 lists of up to 8 rows
constexpr size_t kStaticScratchBytes = kHeadScratchBytes + 2 * kMaxRows * 8 * 4;
static __device__ __align__(256) unsigned char g_head_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
unsigned char* g_scratch_ptr[kMaxDevices];   // device address of g_head_scratch, per device ordinal
int g_sm_count[kMaxDevices];

}  // namespace

extern "C" int ppd_op_head_topk_static(const void* w_packed, int32_t vocab, int32_t K, const float* x, int32_t M,
                                       int32_t ldx, const float* gain, float eps, int32_t k, float* logits,
                                       int32_t* top_ids, float* top_vals, void* stream) {
    if (!w_packed || !x || !logits || !top_ids || !top_vals) return PPD_EINVAL;
    if (vocab < 8 || K < 1 || M < 1 || k < 1) return PPD_EINVAL;
    if (M > kMaxRows || k > PPD_MAX_K) return PPD_ELIMIT;   // the static scratch holds 8 rows x 8 candidates
    if (ldx % kTileCols || ldx < (K + kTileCols - 1) / kTileCols * kTileCols) return PPD_EINVAL;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PPD_ECUDA;
    if (dev < 0 || dev >= kMaxDevices) return PPD_ELIMIT;
    if (!g_scratch_ptr[dev]) {
        // One-time set-up for this device.  In host code `g_head_scratch` is only a handle of the
        // symbol; the address a kernel can use has to be asked for, with this device current.
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_head_scratch) != cudaSuccess || !p) return PPD_ECUDA;
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return PPD_ECUDA;
        g_sm_count[dev] = n;
        g_scratch_ptr[dev] = static_cast<unsigned char*>(p);
    }
    unsigned char* scratch = g_scratch_ptr[dev];
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    // The arrival ticket must start at zero; the array keeps whatever the previous call left.
    if (cudaMemsetAsync(scratch, 0, 256, st) != cudaSuccess) return PPD_ECUDA;
    int* ids8 = reinterpret_cast<int*>(scratch + kHeadScratchBytes);
    float* vals8 = reinterpret_cast<float*>(ids8 + kMaxRows * 8);
    GemvArgs g{};
    g.w = reinterpret_cast<const uint16_t*>(w_packed); g.N = vocab; g.K = K; g.x = x; g.ldx = ldx; g.gain = gain; g.eps = eps;
    g.out = logits; g.ldo = vocab; g.err = nullptr; g.head_scratch = scratch; g.top_ids = ids8; g.top_vals = vals8;
    if (launch_gemv(g, M, kHead, st, false, g_sm_count[dev]) != cudaSuccess) return PPD_ECUDA;
    if (cudaMemcpy2DAsync(top_ids, (size_t)k * 4, ids8, 32, (size_t)k * 4, M, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return PPD_ECUDA;
    if (cudaMemcpy2DAsync(top_vals, (size_t)k * 4, vals8, 32, (size_t)k * 4, M, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return PPD_ECUDA;
    return PPD_OK;
}
