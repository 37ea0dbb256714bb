// Host-side declarations of the kernel launchers (internal to the library).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace ppd {

enum GemvMode : int { kStore = 0, kResid = 1, kSwiglu = 2, kHead = 3 };

struct GemvArgs {
    const uint16_t* w;   // packed weights
    int N, K;            // logical rows / columns
    const float* x;      // [M][ldx]
    int ldx;
    const float* gain;   // [K] or nullptr: RMSNorm fused into the load of x
    float eps;
    const float* resid;  // kResid
    float* out;          // kStore/kResid/kSwiglu: [M][ldo]; kHead: logits [M][ldo]
    int ldo;
    int* err;            // device error word (may be nullptr)
    // kHead only
    void* head_scratch;  // per-CTA candidate lists + ticket
    int* top_ids;        // [M][8]
    float* top_vals;     // [M][8]
};

constexpr int kHeadMaxCtas = 256;
// scratch: ticket (256 B) + [kHeadMaxCtas][8 rows][8] (float, int)
constexpr size_t kHeadScratchBytes = 256 + (size_t)kHeadMaxCtas * 8 * 8 * 8;

// Enqueues the kernel.  pdl: launch with programmatic stream serialization so that the kernel's
// weight prefetch overlaps the tail of the previous kernel in the stream.
cudaError_t launch_gemv(const GemvArgs& a, int M, int mode, cudaStream_t st, bool pdl, int n_sms);

struct AttnArgs {
    const float* qkv;        // [M][3D] un-rotated
    int M, H, hd;
    const int* d_pos;        // device position word or nullptr
    int pos_off;             // rows sit at position p = (d_pos ? *d_pos : 0) + pos_off
    uint16_t* kv_layer;      // this layer's pages: page p = [2][H][64][hd] bf16
    const int* page_table;
    uint16_t* slots;         // branch slots of this layer: row m at slots + m*slot_stride, [2][H][hd]; nullptr = canonical
    long long slot_stride;   // elements
    const float2* rope;      // [pos][hd/2] (cos, sin)
    float* partial;          // split partials [M][H][max_splits][hd + 2]
    int max_splits;
    int* tickets;            // [H] zeroed
    float* out;              // [M][ldo]
    int ldo;
    int* err;
};

cudaError_t launch_attention(const AttnArgs& a, cudaStream_t st, bool pdl, int n_sms);
size_t attn_partial_floats(int M, int H, int hd, int max_splits);

}  // namespace ppd
