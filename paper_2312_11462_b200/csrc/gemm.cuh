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
    // ---- tensor-core path only: the block's rows as three bf16 terms x = b1 + b2 + b3
    __nv_bfloat16* xs = nullptr;         // [3m][K] row-major, row = term * m + r
    bool xs_ready = false;               // false: launch_linear splits X (times gain) into xs first
    float* ssq = nullptr;                // [ssq_cnt][m] pieces of the sums of squares of the rows of X (gain != null)
    int ssq_cnt = 0;                     // entries valid in ssq when xs_ready
    // optional extra outputs for the GEMM that consumes Y next
    __nv_bfloat16* out_xs = nullptr;     // three-term split of (Y * out_gain), [3m][out_ld]
    int out_ld = 0;
    const __nv_bfloat16* out_gain = nullptr;
    float* out_ssq = nullptr;            // [linear_ssq_pieces(...)][m] pieces of the sums of squares of the rows of Y
};

int split_rows(int m);                   // 16, 32, 48 or 64 operand rows hold the 3m terms
int split_ssq_entries(int K);            // ssq pieces the stand-alone split kernel writes

size_t linear_scratch_bytes(int m, int N, int K, bool dual);
int linear_ticket_count(int N);
csd_status launch_linear(const LinearArgs& a, cudaStream_t st);
bool linear_uses_tensor_cores(int m, int N, int K, bool dual);   // the kernel launch_linear would pick (given a.xs)
bool linear_uses_row_ranges(int m, int N, int K, bool dual);     // ... and which of the two tensor-core kernels
int linear_ssq_pieces(int m, int N, int K, bool dual);           // out_ssq pieces that launch writes
int linear_ssq_capacity(int N);                                  // upper bound of the above over m, K

}  // namespace csd
