// Host interface of the block attention over a bf16 K/V cache (defined in attention.cu).
#pragma once
#include "common.cuh"

namespace csd {

struct AttnArgs {
    const float* q = nullptr;             // [m, ldq] fp32; head h occupies columns h*Dh .. h*Dh+Dh-1
    int ldq = 0, m = 0;
    const __nv_bfloat16* Kc = nullptr;    // [H][cap][Dh]
    const __nv_bfloat16* Vc = nullptr;
    int cap = 0, H = 0, Dh = 0;
    int n_keys = 0;                       // keys visible to row 0 (causal: row r sees n_keys + r)
    int causal = 0;
    float scale = 1.f;
    const float* bias = nullptr;          // optional [H][bias_len], indexed by (key - query) + bias_zero
    int bias_len = 0, bias_zero = 0;
    int q_pos0 = 0;                       // position of row 0 (for the bias)
    float* out = nullptr;                 // [m, ldo]
    int ldo = 0;
    __nv_bfloat16* out_xs = nullptr;      // optional: the output rows as three bf16 terms, row = term * m + r
    int out_xs_ld = 0;
    float* partial = nullptr;             // split scratch (attn_scratch_bytes)
    unsigned* tickets = nullptr;          // H zero-initialised words
    int max_keys = 0;                     // capacity used to size the scratch
};

int attn_splits(int total_keys, int H);
size_t attn_scratch_bytes(int max_keys, int H, int Dh);
csd_status launch_attention(const AttnArgs& a, cudaStream_t st);

}  // namespace csd
