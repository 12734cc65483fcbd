// Weight-streaming skinny GEMM  Y[m, N] = X[m, K] . W[N, K]^T  for m <= 17 rows.
//
// Every bf16 weight is read from HBM exactly once with 128-bit streaming loads and used for m
// fused multiply-adds on the CUDA cores (fp32 accumulation), so for small m the kernel is bound
// by HBM bandwidth.  Work is cut into units of (TN output columns) x (one K slice); a CTA takes
// one unit, keeps its X slice in shared memory, and each warp streams R weight rows at a time.
// With more than one K slice the CTAs leave fp32 partial tiles in scratch and the CTA that
// arrives last at the tile's ticket adds them in slice order (deterministic) and runs the
// epilogue (store / residual add / gated activation, optional RMS-norm scaling).  No CTA ever
// waits for another.
#include "gemm.cuh"

namespace csd {

constexpr int GT = 256;          // threads per CTA
constexpr int GW = GT / 32;      // warps per CTA
constexpr int KSTEP = 256;       // K elements one warp covers per step (32 lanes x 8 bf16)

template <int M, bool DUAL>
struct RowsPerWarp {
    static constexpr int value = DUAL ? (M <= 5 ? 4 : (M <= 9 ? 2 : 1)) : (M <= 9 ? 4 : 2);
};

struct LinearPlan {
    int R, TN, ntiles, steps_total, steps_per, kslices, KSP;
    size_t smem, unit_floats;
};

static int rows_per_warp(int m, bool dual) {
    return dual ? (m <= 5 ? 4 : (m <= 9 ? 2 : 1)) : (m <= 9 ? 4 : 2);
}

static LinearPlan plan_linear(int m, int N, int K, bool dual) {
    LinearPlan p;
    p.R = rows_per_warp(m, dual);
    p.TN = GW * p.R;
    p.ntiles = (N + p.TN - 1) / p.TN;
    p.steps_total = (K + KSTEP - 1) / KSTEP;
    int max_steps = (56 * 1024) / (m * KSTEP * 4);       // X slice of at most 56 KB
    if (max_steps < 1) max_steps = 1;
    int kslices = (p.steps_total + max_steps - 1) / max_steps;
    const int want_units = 148 * 6;
    int by_units = (want_units + p.ntiles - 1) / p.ntiles;
    if (by_units > kslices) kslices = by_units;
    int min_steps = 2;                                    // keep at least two steps per slice
    int cap = p.steps_total / min_steps;
    if (cap < 1) cap = 1;
    if (kslices > cap) kslices = cap;
    int need = (p.steps_total + max_steps - 1) / max_steps;
    if (kslices < need) kslices = need;
    p.steps_per = (p.steps_total + kslices - 1) / kslices;
    p.kslices = (p.steps_total + p.steps_per - 1) / p.steps_per;
    p.KSP = p.steps_per * KSTEP;
    p.unit_floats = (size_t)(dual ? 2 : 1) * m * p.TN + m;
    p.smem = ((size_t)m * p.KSP + (size_t)(dual ? 2 : 1) * m * p.TN + m + 8) * sizeof(float);
    return p;
}

struct GemmParams {
    const __nv_bfloat16* W;
    const __nv_bfloat16* W2;
    const float* X;
    const __nv_bfloat16* gain;
    float* Y;
    float* partial;
    unsigned* tickets;
    int N, K, ldx, ldy, m;
    int steps_per, kslices, KSP, ntiles;
    int epilogue;
    float eps;
};

__device__ __forceinline__ float gelu_tanh_f(float x) {
    return 0.5f * x * (1.f + tanhf(0.7978845608028654f * (x + 0.044715f * x * x * x)));
}
__device__ __forceinline__ float silu_f(float x) { return x / (1.f + __expf(-x)); }

__device__ __forceinline__ float dot8(const uint4& w, const float4& a, const float4& b, float acc) {
    acc = fmaf(bf16lo(w.x), a.x, acc);
    acc = fmaf(bf16hi(w.x), a.y, acc);
    acc = fmaf(bf16lo(w.y), a.z, acc);
    acc = fmaf(bf16hi(w.y), a.w, acc);
    acc = fmaf(bf16lo(w.z), b.x, acc);
    acc = fmaf(bf16hi(w.z), b.y, acc);
    acc = fmaf(bf16lo(w.w), b.z, acc);
    acc = fmaf(bf16hi(w.w), b.w, acc);
    return acc;
}

template <int M, bool DUAL>
__global__ void __launch_bounds__(GT)
skinny_gemm_kernel(const GemmParams p) {
    constexpr int R = RowsPerWarp<M, DUAL>::value;
    constexpr int TN = GW * R;
    constexpr int NT = DUAL ? 2 : 1;
    extern __shared__ __align__(16) float smem[];
    float* xs = smem;                           // [M][KSP], each 256-step stored as [half][lane][4]
    float* tile = xs + (size_t)M * p.KSP;       // [NT][M][TN]
    float* ss = tile + NT * M * TN;             // [M] sum of squares of this K slice
    __shared__ int s_last;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int ntile = blockIdx.x / p.kslices, ks = blockIdx.x % p.kslices;
    const int k0 = ks * p.KSP;
    const int k1 = min(p.K, k0 + p.KSP);
    const int kw = k1 - k0;
    const int steps = (kw + KSTEP - 1) / KSTEP;

    // ---- stage the X slice (times the norm gain) into shared memory, permuted for
    //      conflict-free 128-bit reads: k = s*256 + lane*8 + h*4 + i  ->  s*256 + h*128 + lane*4 + i
    for (int idx = tid; idx < M * steps * KSTEP; idx += GT) {
        const int r = idx / (steps * KSTEP), kk = idx % (steps * KSTEP);
        float v = 0.f;
        if (r < p.m && kk < kw) {
            v = p.X[(size_t)r * p.ldx + k0 + kk];
            if (p.gain) v *= __bfloat162float(p.gain[k0 + kk]);
        }
        const int s = kk >> 8, o = kk & 255;
        const int pos = (s << 8) + (((o >> 2) & 1) << 7) + ((o >> 3) << 2) + (o & 3);
        xs[(size_t)r * p.KSP + pos] = v;
    }
    if (p.gain) {
        for (int r = warp; r < M; r += GW) {
            float a = 0.f;
            if (r < p.m)
                for (int kk = lane; kk < kw; kk += 32) {
                    float v = p.X[(size_t)r * p.ldx + k0 + kk];
                    a = fmaf(v, v, a);
                }
            a = warp_sum(a);
            if (lane == 0) ss[r] = a;
        }
    }
    __syncthreads();

    // ---- stream R weight rows per warp
    const int n_base = ntile * TN + warp * R;
    const __nv_bfloat16* wrow[NT][R];
#pragma unroll
    for (int rr = 0; rr < R; ++rr) {
        int n = n_base + rr;
        if (n >= p.N) n = p.N - 1;              // clamped rows are loaded but never stored
        wrow[0][rr] = p.W + (size_t)n * p.K + k0 + lane * 8;
        if (DUAL) wrow[NT - 1][rr] = p.W2 + (size_t)n * p.K + k0 + lane * 8;
    }
    float acc[NT][R][M];
#pragma unroll
    for (int t = 0; t < NT; ++t)
#pragma unroll
        for (int rr = 0; rr < R; ++rr)
#pragma unroll
            for (int r = 0; r < M; ++r) acc[t][rr][r] = 0.f;

    uint4 wcur[NT][R], wnext[NT][R];
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int t = 0; t < NT; ++t)
#pragma unroll
        for (int rr = 0; rr < R; ++rr) wcur[t][rr] = (lane * 8 < kw) ? ldg_stream(wrow[t][rr]) : zero4;

    for (int s = 0; s < steps; ++s) {
        const int knext = (s + 1) * KSTEP + lane * 8;
#pragma unroll
        for (int t = 0; t < NT; ++t)
#pragma unroll
            for (int rr = 0; rr < R; ++rr)
                wnext[t][rr] = (s + 1 < steps && knext < kw) ? ldg_stream(wrow[t][rr] + (s + 1) * KSTEP) : zero4;
        const float* xp = xs + (s << 8) + lane * 4;
#pragma unroll
        for (int r = 0; r < M; ++r) {
            const float4 xa = *reinterpret_cast<const float4*>(xp + (size_t)r * p.KSP);
            const float4 xb = *reinterpret_cast<const float4*>(xp + (size_t)r * p.KSP + 128);
#pragma unroll
            for (int t = 0; t < NT; ++t)
#pragma unroll
                for (int rr = 0; rr < R; ++rr) acc[t][rr][r] = dot8(wcur[t][rr], xa, xb, acc[t][rr][r]);
        }
#pragma unroll
        for (int t = 0; t < NT; ++t)
#pragma unroll
            for (int rr = 0; rr < R; ++rr) wcur[t][rr] = wnext[t][rr];
    }

    // ---- reduce over lanes, gather the CTA's tile in shared memory
#pragma unroll
    for (int t = 0; t < NT; ++t)
#pragma unroll
        for (int rr = 0; rr < R; ++rr)
#pragma unroll
            for (int r = 0; r < M; ++r) {
                float v = warp_sum(acc[t][rr][r]);
                if (lane == 0) tile[(t * M + r) * TN + warp * R + rr] = v;
            }
    __syncthreads();

    constexpr int UNIT = NT * M * TN;
    if (p.kslices > 1) {
        float* mine = p.partial + ((size_t)ntile * p.kslices + ks) * (UNIT + M);
        for (int i = tid; i < UNIT; i += GT) mine[i] = tile[i];
        if (p.gain && tid < M) mine[UNIT + tid] = ss[tid];
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            unsigned old = atomicAdd(&p.tickets[ntile], 1u);
            s_last = (old == (unsigned)p.kslices - 1u);
            if (s_last) p.tickets[ntile] = 0u;     // ready for the next launch
        }
        __syncthreads();
        if (!s_last) return;
        __threadfence();
        const float* all = p.partial + (size_t)ntile * p.kslices * (UNIT + M);
        for (int i = tid; i < UNIT + M; i += GT) {
            if (i >= UNIT && !p.gain) break;
            float v = 0.f;
            for (int c = 0; c < p.kslices; ++c) v += __ldcg(all + (size_t)c * (UNIT + M) + i);
            if (i < UNIT) tile[i] = v; else ss[i - UNIT] = v;
        }
        __syncthreads();
    }

    // ---- epilogue
    for (int i = tid; i < M * TN; i += GT) {
        const int r = i / TN, c = i % TN;
        const int n = ntile * TN + c;
        if (r >= p.m || n >= p.N) continue;
        float v = tile[r * TN + c];
        float scale = 1.f;
        if (p.gain) scale = rsqrtf(ss[r] / (float)p.K + p.eps);
        v *= scale;
        if (DUAL) {
            float u = tile[(M + r) * TN + c] * scale;
            v = (p.epilogue == EPI_GEGLU ? gelu_tanh_f(v) : silu_f(v)) * u;
        }
        float* y = p.Y + (size_t)r * p.ldy + n;
        if (p.epilogue == EPI_ADD) *y += v; else *y = v;
    }
}

template <int M, bool DUAL>
static csd_status launch_one(const GemmParams& gp, const LinearPlan& pl, cudaStream_t st) {
    auto kern = skinny_gemm_kernel<M, DUAL>;
    static bool attr_set = false;   // per instantiation
    if (!attr_set) {
        CSD_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024));
        attr_set = true;
    }
    kern<<<(unsigned)(pl.ntiles * pl.kslices), GT, pl.smem, st>>>(gp);
    count_launch();
    CSD_CUDA(cudaGetLastError());
    return CSD_OK;
}

size_t linear_scratch_bytes(int m, int N, int K, bool dual) {
    size_t worst = 0;
    for (int mm = 1; mm <= m; ++mm) {
        LinearPlan pl = plan_linear(mm, N, K, dual);
        size_t b = pl.kslices > 1 ? (size_t)pl.ntiles * pl.kslices * pl.unit_floats * sizeof(float) : 0;
        if (b > worst) worst = b;
    }
    return align_up(worst, 256);
}

int linear_ticket_count(int N) { return (N + GW - 1) / GW + 1; }   // TN >= GW columns per tile

csd_status launch_linear(const LinearArgs& a, cudaStream_t st) {
    if (!a.W || !a.X || !a.Y || a.m < 1 || a.m > CSD_MAX_ROWS || a.N < 1 || a.K < 8 || (a.K & 7))
        return CSD_ERR_INVALID_ARG;
    const bool dual = a.W2 != nullptr;
    if (dual != (a.epilogue == EPI_SWIGLU || a.epilogue == EPI_GEGLU)) return CSD_ERR_INVALID_ARG;
    if ((((uintptr_t)a.W) & 15) || (dual && (((uintptr_t)a.W2) & 15))) return CSD_ERR_INVALID_ARG;
    const LinearPlan pl = plan_linear(a.m, a.N, a.K, dual);
    if (pl.kslices > 1 && (!a.partial || !a.tickets)) return CSD_ERR_INVALID_ARG;
    GemmParams gp;
    gp.W = a.W; gp.W2 = a.W2; gp.X = a.X; gp.gain = a.gain; gp.Y = a.Y; gp.partial = a.partial;
    gp.tickets = a.tickets; gp.N = a.N; gp.K = a.K; gp.ldx = a.ldx; gp.ldy = a.ldy; gp.m = a.m;
    gp.steps_per = pl.steps_per; gp.kslices = pl.kslices; gp.KSP = pl.KSP; gp.ntiles = pl.ntiles;
    gp.epilogue = a.epilogue; gp.eps = a.eps;
#define CSD_CASE(MM)                                                              \
    case MM:                                                                      \
        return dual ? launch_one<MM, true>(gp, pl, st) : launch_one<MM, false>(gp, pl, st);
    switch (a.m) {
        CSD_CASE(1) CSD_CASE(2) CSD_CASE(3) CSD_CASE(4) CSD_CASE(5) CSD_CASE(6) CSD_CASE(7) CSD_CASE(8)
        CSD_CASE(9) CSD_CASE(10) CSD_CASE(11) CSD_CASE(12) CSD_CASE(13) CSD_CASE(14) CSD_CASE(15)
        CSD_CASE(16) CSD_CASE(17)
    }
#undef CSD_CASE
    return CSD_ERR_INVALID_ARG;
}

}  // namespace csd

using namespace csd;

extern "C" size_t csd_linear_workspace_bytes(int m, int N, int K) {
    if (m < 1 || m > CSD_MAX_ROWS || N < 1 || K < 8) return 0;
    return linear_scratch_bytes(m, N, K, false) + align_up((size_t)linear_ticket_count(N) * sizeof(unsigned), 256);
}

// The ticket words at the start of the workspace must be zero before the first call; every
// launch leaves them zero again, so one cudaMemset after allocation is enough.
extern "C" csd_status csd_linear(const void* W_bf16_dev, int N, int K, const float* X_dev, int m, float* Y_dev,
                                 void* workspace_dev, size_t workspace_bytes, void* stream) {
    if (m < 1 || m > CSD_MAX_ROWS || N < 1 || K < 8 || (K & 7)) return CSD_ERR_INVALID_ARG;
    if (!W_bf16_dev || !X_dev || !Y_dev) return CSD_ERR_INVALID_ARG;
    size_t need = csd_linear_workspace_bytes(m, N, K);
    if (workspace_bytes < need || (need && !workspace_dev)) return CSD_ERR_CAPACITY;
    if (((uintptr_t)workspace_dev) & 255) return CSD_ERR_INVALID_ARG;
    size_t toff = align_up((size_t)linear_ticket_count(N) * sizeof(unsigned), 256);
    LinearArgs a;
    a.W = (const __nv_bfloat16*)W_bf16_dev; a.N = N; a.K = K; a.X = X_dev; a.ldx = K; a.m = m;
    a.Y = Y_dev; a.ldy = N; a.epilogue = EPI_STORE;
    a.tickets = (unsigned*)workspace_dev;
    a.partial = (float*)((char*)workspace_dev + toff);
    return launch_linear(a, (cudaStream_t)stream);
}
