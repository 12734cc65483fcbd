// Host interface of the tensor-core (tcgen05 + TMA) variant of the skinny GEMM (gemm_tc.cu).
#pragma once
#include "gemm.cuh"

namespace csd {

int tc_sm_count();
bool tc_supported(int m, int N, int K, bool dual);
size_t tc_scratch_bytes(int m, int N, int K, bool dual);
int tc_ticket_count(int N);
csd_status launch_linear_tc(const LinearArgs& a, cudaStream_t st);
csd_status launch_split_rows(const LinearArgs& a, cudaStream_t st);   // a.X (times a.gain) -> a.xs, a.ssq

// row-range variant (gemm_rs.cu): every CTA owns whole output columns, nothing is shared between CTAs
bool rs_supported(int m, int N, int K, bool dual);
int rs_ssq_pieces(int m, int N, int K, bool dual);     // sum-of-squares pieces its epilogue writes
int rs_box_rows(int m, int N, int K, bool dual);       // weight rows per CTA and range
csd_status launch_linear_rs(const LinearArgs& a, cudaStream_t st);

// wide-block variant (gemm_wide.cu): up to CSD_WIDE_ROWS rows per pass, two bf16 terms per value
constexpr int CSD_WIDE_ROWS = 128;
struct WideArgs {
    const __nv_bfloat16* W = nullptr;    // [N, K] row-major
    const __nv_bfloat16* W2 = nullptr;   // gated feed-forward only
    int N = 0, K = 0, m = 0;
    const __nv_bfloat16* xs = nullptr;   // the rows as two bf16 terms [2][mpad][K], mpad = m rounded up to 16
    const float* ssq = nullptr;          // with an RMS norm: pieces [ssq_cnt][m] of the rows' sums of squares
    int ssq_cnt = 0;
    float eps = 0.f;
    float* Y = nullptr;                  // [m, ldy]
    int ldy = 0, epilogue = EPI_STORE;
    __nv_bfloat16* out_xs = nullptr;     // optional: (Y * out_gain) in two-term form [2][mpad][out_ld] for the next wide GEMM
    int out_ld = 0;
    const __nv_bfloat16* out_gain = nullptr;
    float* out_ssq = nullptr;            // optional: [wide_ssq_pieces(...)][m] pieces of the sums of squares of the rows of Y
    float* partial = nullptr;            // scratch of wide_partial_bytes(...) for K-partitioned launches (optional)
};
bool wide_supported(int m, int N, int K, bool dual);
int wide_ssq_pieces(int m, int N, int K, bool dual);
int wide_ssq_capacity(int N);
size_t wide_partial_bytes(int m, int N, int K, bool dual);
int wide_split_pieces(int K);
csd_status launch_wide_split(const float* X, int ldx, int K, int m, const __nv_bfloat16* gain, __nv_bfloat16* xs,
                             float* ssq, cudaStream_t st);
csd_status launch_linear_wide(const WideArgs& a, cudaStream_t st);

// 0 = automatic choice, 1 = CUDA-core kernel only, 2 = stream-K tensor-core kernel wherever it applies,
// 3 = row-range tensor-core kernel wherever it applies (stream-K elsewhere)
void set_gemm_path(int path);
int gemm_path();

}  // namespace csd
