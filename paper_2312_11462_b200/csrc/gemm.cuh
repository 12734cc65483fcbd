// Host interface of the weight-streaming skinny GEMM (defined in gemm.cu).
#pragma once
#include "common.cuh"

namespace csd {

enum : int { EPI_STORE = 0, EPI_ADD = 1, EPI_SWIGLU = 2, EPI_GEGLU = 3 };

struct LinearArgs {
    const __nv_bfloat16* W = nullptr;    // [N, K] row-major
    const __nv_bfloat16* W2 = nullptr;   // gated feed-forward only: the "up" matrix, same shape
    int N = 0, K = 0;
    const float* X = nullptr;            // [m, ldx]
    int ldx = 0, m = 0;
    const __nv_bfloat16* gain = nullptr; // RMS-norm gain [K]: Y = rstd(x) * ((x * gain) . W^T)
    float eps = 0.f;
    float* Y = nullptr;                  // [m, ldy]
    int ldy = 0;
    int epilogue = EPI_STORE;
    float* partial = nullptr;            // split-K scratch (linear_scratch_bytes)
    unsigned* tickets = nullptr;         // zero-initialised, linear_ticket_count entries
};

size_t linear_scratch_bytes(int m, int N, int K, bool dual);
int linear_ticket_count(int N);
csd_status launch_linear(const LinearArgs& a, cudaStream_t st);

}  // namespace csd
