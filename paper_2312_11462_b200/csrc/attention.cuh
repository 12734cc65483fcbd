// Host interface of the block attention over a bf16 K/V cache (defined in attention.cu).
#pragma once
#include "common.cuh"

namespace csd {

struct AttnArgs {
    const float* q = nullptr;             // [m, ldq] fp32; head h occupies columns h*Dh .. h*Dh+Dh-1
    int ldq = 0, m = 0;
    __nv_bfloat16* Kc = nullptr;          // [H][cap][Dh]
    __nv_bfloat16* Vc = nullptr;
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
    int out_xs_rows = 0;                  // rows per term of the out_xs buffer (0: m) and this block's first row in it
    int out_xs_row0 = 0;
    // Self-attention of a drafted block (causal, n_keys = committed keys + 1): the block's own key
    // and value rows are still fp32 projections [m, ld_new]; the kernel rotates q and k (when
    // rope tables [pos][Dh/2] are given), rounds k and v to bf16, appends them to the cache at
    // positions n_keys-1 .. n_keys+m-2 and attends over committed and new rows alike.
    const float* k_new = nullptr;
    const float* v_new = nullptr;
    int ld_new = 0;
    const float* rope_cos = nullptr;
    const float* rope_sin = nullptr;
    // true when every cache row this call reads (other than the block's own) was complete before
    // the kernel right before this one on the stream began; the tile requests then go out before
    // the dependency wait
    bool kv_settled = false;
    // tree-shaped block (host arrays of m entries, copied into the launch): bit j of tree_mask[r] set
    // when row r may see block row j; tree_depth[r] = number of ancestors of row r inside the block.
    // Null: the block is a chain (row r sees rows 0..r).
    const unsigned* tree_mask = nullptr;
    const int* tree_depth = nullptr;
};

int attn_splits(int total_keys, int H);
void set_attention_cuda_cores(bool on);   // true: always the CUDA-core kernel (for comparison runs)
csd_status launch_attention(const AttnArgs& a, cudaStream_t st);

}  // namespace csd
