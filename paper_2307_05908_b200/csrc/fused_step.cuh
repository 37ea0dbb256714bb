// Persistent decode-step kernel: one launch runs a whole greedy or PPD step (internal header).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace ppd {

// indices into the device state block (32-bit words); the barrier counter is a 64-bit word
enum StateWord : int {
    S_POS = 0, S_PENDING = 1, S_STEP = 2, S_TICKET = 3, S_LAST_TOKEN = 4, S_LAST_HIT = 5, S_ERR = 6,
    S_PREV_HIT = 7, S_PREV_B = 8, S_HEAD_TICKET = 9,
    S_BAR_COUNT = 16,  // u64: grid-barrier arrivals since the context was created
    S_BAR_BASE = 18,   // u64: value of the counter when the next launch starts
};

struct LaneBuf {          // activation workspace of one lane (main: 1 row; branch: up to 8 rows)
    float *h, *qkv, *attn, *z, *partial;
    int* tickets;         // [H], zero between launches
};

enum StepMode : int { kPrefillToken = 0, kGreedyStep = 1, kPpdStep = 2 };

struct FusedArgs {
    // model
    int d, D, F, V, H, hd, Dp, Fp;
    float eps;
    const uint8_t* layers;
    long long layer_bytes, off_wqkv, off_wo, off_wgu, off_wd, off_g1, off_g2;
    const uint16_t* emb;
    const float* g_final;
    const uint16_t* w_head;
    const uint16_t* w_head_early;   // classifier of the early head (== w_head unless one was loaded)
    // KV cache
    uint16_t* kv;
    long long kv_layer_elems;
    const int* page_table;
    uint16_t* slots;
    long long slot_stride, slot_layer_stride;
    const float2* rope;
    int max_splits;
    LaneBuf main, br;
    // program
    int mode;              // StepMode
    int k, l;              // PPD: candidates, early layer
    const int* token_src;  // kPrefillToken: the token to run; otherwise state[S_PENDING] is used
    int pos_val;           // kPrefillToken: its position
    // heads
    float *logits_early, *logits_final;
    int *top_early, *top_final;   // ids[8]; values (float) at +32 words
    void* head_scratch;
    // state and outputs
    int* state;
    int* out_tokens;
    uint8_t* out_hit;
    float* out_margin;
    unsigned long long* timeline;   // optional: [cta in {0, last}][phase][start, end] in ns; nullptr = off
    int timeline_phases;            // capacity in phases
};

// Launches the step kernel for `mb` branch rows (0 = no branches: prefill token or greedy step).
cudaError_t launch_fused_step(const FusedArgs& a, int mb, cudaStream_t st, bool pdl, int n_sms);

}  // namespace ppd
