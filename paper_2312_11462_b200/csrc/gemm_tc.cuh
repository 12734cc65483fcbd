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

// 0 = automatic choice, 1 = CUDA-core kernel only, 2 = stream-K tensor-core kernel wherever it applies,
// 3 = row-range tensor-core kernel wherever it applies (stream-K elsewhere)
void set_gemm_path(int path);
int gemm_path();

}  // namespace csd
