// A chain of dependent skinny GEMMs in ONE persistent kernel (for example attention-output
// projection -> gated feed-forward -> down projection -> next layer's q|k|v projection).
//
// Each GEMM is the tensor-core contraction of gemm_tc.cu (TMA-staged 128 x 64 weight tiles,
// tcgen05.mma, three-term bf16 rows, equal contiguous shares of (tile, K block) units per CTA,
// ticketed fix-up of straddling tiles).  What the chain adds: the TMA producer keeps requesting
// weight tiles of the NEXT GEMM while the current one drains (weights depend on nothing), so the
// 12-stage ring is full when the dependency resolves and the SMs never stop streaming; only the
// rows' terms (a 2-8 KB tile per stage, written by the previous GEMM's epilogue) wait until every
// CTA has reported that GEMM finished.  That report is a counter in global memory which CTAs
// poll a bounded number of times; the kernel is launched cooperatively (one CTA per SM, all
// resident), so the wait always ends, and if it ever did not the CTA records CSD_ERR_TIMEOUT,
// stops, frees its tensor memory and returns.
#include "gemm_tc.cuh"
#include "tc_common.cuh"

namespace csd {

constexpr int CHAIN_MAX_OPS = 4;
constexpr size_t CHAIN_SMEM = 224 * 1024;      // one CTA per SM
constexpr int DEP_POLL_LIMIT = 4000000;

struct alignas(64) ChainOpDev {
    CUtensorMap tmW, tmW2, tmX;
    float* Y; const float* ssq_in; __nv_bfloat16* out_xs; const __nv_bfloat16* out_gain; float* out_ssq;
    unsigned* tickets;
    int ssq_cnt, out_ld, N, K, ldy, nkb, tiles, epilogue, dual;
    float eps;
};

struct alignas(64) ChainParams {
    ChainOpDev op[CHAIN_MAX_OPS];
    float* partial; unsigned* done; int* status;
    unsigned done_target;          // value every done[j] reaches when all CTAs have finished GEMM j
    int n_ops, stages;
};

struct __align__(8) ChainCtrl {
    uint64_t full[12], empty[12], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    int abort_flag, last_flag;
    float scale[32];
};

__device__ __forceinline__ float ch_gelu(float x) {
    return 0.5f * x * (1.f + tanhf(0.7978845608028654f * (x + 0.044715f * x * x * x)));
}
__device__ __forceinline__ float ch_silu(float x) { return x / (1.f + expf(-x)); }

__device__ __forceinline__ unsigned ch_unit_begin(unsigned c, unsigned units, unsigned ctas) { return c * units / ctas; }
__device__ __forceinline__ int ch_cta_of_unit(unsigned u, unsigned units, unsigned ctas) {
    unsigned c = ((u + 1) * ctas - 1) / units;
    while (c + 1 < ctas && ch_unit_begin(c + 1, units, ctas) <= u) ++c;
    while (c > 0 && ch_unit_begin(c, units, ctas) > u) --c;
    return (int)c;
}
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {   // one poll, no spinning
    uint32_t ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// where a unit of GEMM `o` lives: tile, K block, and (gated feed-forward) which of the two matrices
struct UnitPos { int tile, kb, which; };
__device__ __forceinline__ UnitPos unit_pos(const ChainOpDev& o, unsigned u) {
    const int per_tile = o.nkb * (o.dual ? 2 : 1);
    UnitPos p;
    p.tile = (int)(u / per_tile);
    const int rem = (int)(u % per_tile);
    p.kb = o.dual ? rem >> 1 : rem;
    p.which = o.dual ? rem & 1 : 0;
    return p;
}
