// Model handle shared by model.cu and cascade.cu.
#pragma once
#include <vector>
#include "attention.cuh"
#include "common.cuh"
#include "gemm.cuh"
#include "gemm_tc.cuh"

namespace csd {
struct LayerW {
    const __nv_bfloat16 *norm1, *wq, *wk, *wv, *wo, *norm_x, *xq, *xk, *xv, *xo, *norm2, *wgate, *wup, *wdown;
};
}  // namespace csd

struct csd_model {
    csd_model_config cfg;
    int di = 0;                 // n_heads * d_head
    int enc_len = 0;            // encoder positions cached by csd_encoder_forward
    const __nv_bfloat16 *embed = nullptr, *final_norm = nullptr, *lm_head = nullptr, *enc_rel_bias = nullptr,
                        *dec_rel_bias = nullptr, *enc_final_norm = nullptr;
    std::vector<csd::LayerW> enc, dec;
    // workspace views
    __nv_bfloat16 *kcache = nullptr, *vcache = nullptr;   // [layer][head][max_seq][Dh]
    __nv_bfloat16 *xk = nullptr, *xv = nullptr;           // cross K/V [layer][head][max_enc_len][Dh]
    __nv_bfloat16 *ek = nullptr, *ev = nullptr;           // encoder self K/V of the layer in flight
    size_t layer_kv = 0, layer_x = 0;
    float *x = nullptr, *qkv = nullptr, *attn = nullptr, *act = nullptr, *xenc = nullptr, *qkv_enc = nullptr;
    float *rope_c = nullptr, *rope_s = nullptr, *dec_bias = nullptr, *enc_bias = nullptr;
    float* gemm_partial = nullptr;
    unsigned* gemm_tickets = nullptr;
    __nv_bfloat16* xs_tmp = nullptr;    // three-term bf16 split of a GEMM's input rows (tensor-core path)
    float* ssq_tmp = nullptr;           // pieces of the rows' sums of squares written with it
    // activations handed from kernel to kernel in three-term form (tensor-core path)
    __nv_bfloat16 *xs_x = nullptr, *xs_attn = nullptr, *xs_act = nullptr;   // [3*17][d], [3*17][d_inner], [3*17][d_ff]
    float* ssq_x = nullptr;             // [ssq_x_cnt][rows] pieces of the sums of squares of the residual rows
    int ssq_x_cnt = 0;                  // pieces the GEMM that last produced the residual rows wrote
    int* status = nullptr;
    // wide blocks (prompt prefill, encoder pass): up to CSD_WIDE_ROWS rows per pass over the weights
    bool wide = false;                  // every layer matrix takes the wide-block kernel
    float *wx = nullptr, *wqkv = nullptr, *wattn = nullptr, *wact = nullptr;            // [128][d], [128][3 d_inner], ...
    __nv_bfloat16 *wxs_x = nullptr, *wxs_attn = nullptr, *wxs_act = nullptr;            // two-term rows [2][128][K]
    float* wssq = nullptr;              // pieces of the rows' sums of squares
    float* wpart = nullptr;             // partial planes of K-partitioned wide GEMMs
    // optional per-kernel-class timing (csd_model_profile): event pairs around every launch
    bool prof = false;
    std::vector<cudaEvent_t> prof_ev;      // start, stop, start, stop, ...
    std::vector<int> prof_kind;            // class of each pair: 0 GEMM, 1 attention, 2 other
    size_t prof_used = 0;                  // pairs recorded since the last read
    double prof_gemm_bytes = 0.0;          // weight bytes the recorded GEMM launches streamed
};

namespace csd {
// Records an event pair around the launches made during its lifetime when profiling is on.
struct ProfScope {
    csd_model* M; cudaStream_t st; bool on;
    ProfScope(csd_model* m, int kind, cudaStream_t s) : M(m), st(s), on(m->prof) {
        if (!on) return;
        if (M->prof_used * 2 + 2 > M->prof_ev.size()) {
            cudaEvent_t a = nullptr, b = nullptr;
            if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { on = false; return; }
            M->prof_ev.push_back(a); M->prof_ev.push_back(b); M->prof_kind.push_back(kind);
        }
        M->prof_kind[M->prof_used] = kind;
        cudaEventRecord(M->prof_ev[M->prof_used * 2], st);
    }
    ~ProfScope() {
        if (!on) return;
        cudaEventRecord(M->prof_ev[M->prof_used * 2 + 1], st);
        M->prof_used += 1;
    }
};
}  // namespace csd
