// Weight-streaming skinny GEMM  Y[m, N] = X[m, K] . W[N, K]^T  for m <= 17 rows.
//
// Every bf16 weight is read from HBM exactly once with 128-bit streaming loads and used for m
// fused multiply-adds on the CUDA cores (fp32 accumulation), so for small m the kernel is bound
// by HBM bandwidth.  The grid is persistent (two CTAs per SM).  A CTA owns one K slice, keeps
// that slice of X in shared memory for its whole life, and its warps walk over groups of R
// weight rows with a register double buffer that keeps loads in flight across groups; warps
// never synchronise with each other after the X slice is staged.  With more than one K slice
// a warp leaves its fp32 partial sums in scratch and the warp that arrives last at the group's
// ticket adds them in slice order (deterministic) and runs the epilogue (store / residual add /
// gated activation, optional RMS-norm scaling).  Nothing ever waits for another CTA.  The first
// weight loads are issued before the programmatic-dependent-launch wait, so they overlap the
// tail of the kernel that produces X.
#include "gemm_tc.cuh"

namespace csd {

constexpr int GT = 256;          // threads per CTA
constexpr int GW = GT / 32;      // warps per CTA
constexpr int KSTEP = 256;       // K elements one warp covers per step (32 lanes x 8 bf16)
constexpr int CTAS_PER_SM = 2;
constexpr long long AUTO_TC_MIN_WEIGHTS = 1 << 20;   // automatic choice: matrices at least this large go to the tensor-core kernel
constexpr size_t SMEM_BUDGET = 110 * 1024;   // per CTA, so that two CTAs share an SM

template <int M, bool DUAL>
struct RowsPerWarp {
    static constexpr int value = DUAL ? (M <= 9 ? 2 : 1) : (M <= 9 ? 4 : 2);
};

struct LinearPlan {
    int R, NV, groups, steps_total, steps_per, kslices, KSP, grid;
    size_t smem, scratch_floats;
};

static int rows_per_warp(int m, bool dual) {
    return dual ? (m <= 9 ? 2 : 1) : (m <= 9 ? 4 : 2);
}

static int sm_count() {
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
    }
    return n;
}

static LinearPlan plan_linear(int m, int N, int K, bool dual) {
    LinearPlan p;
    p.R = rows_per_warp(m, dual);
    p.NV = (dual ? 2 : 1) * p.R * m;                       // partial sums one warp produces per row group
    p.groups = (N + p.R - 1) / p.R;
    p.steps_total = (K + KSTEP - 1) / KSTEP;
    const size_t red = (size_t)GW * p.NV * 33 * sizeof(float) + 64 * sizeof(float);
    int kslices = 1;
    for (;; ++kslices) {
        int per = (p.steps_total + kslices - 1) / kslices;
        if ((size_t)m * per * KSTEP * sizeof(float) + red <= SMEM_BUDGET || per == 1) break;
    }
    p.steps_per = (p.steps_total + kslices - 1) / kslices;
    p.kslices = (p.steps_total + p.steps_per - 1) / p.steps_per;
    p.KSP = p.steps_per * KSTEP;
    p.smem = (size_t)m * p.KSP * sizeof(float) + red;
    // persistent grid: every SM gets CTAS_PER_SM CTAs, a multiple of the slice count, and no more
    // warps per slice than there are row groups
    int grid = sm_count() * CTAS_PER_SM;
    int need = ((p.groups + GW - 1) / GW) * p.kslices;
    if (grid > need) grid = need;
    grid = (grid / p.kslices) * p.kslices;
    if (grid < p.kslices) grid = p.kslices;
    p.grid = grid;
    p.scratch_floats = p.kslices > 1 ? (size_t)p.kslices * p.groups * p.NV + (size_t)p.kslices * m : 0;
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
    int steps_per, kslices, KSP, groups;
    int epilogue;
    float eps;
};

__device__ __forceinline__ float gelu_tanh_f(float x) {
    return 0.5f * x * (1.f + tanhf(0.7978845608028654f * (x + 0.044715f * x * x * x)));
}
__device__ __forceinline__ float silu_f(float x) { return x / (1.f + expf(-x)); }

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

// Programmatic dependent launch: the weights do not depend on the previous kernel, so a CTA may
// start streaming them before the producer of X has finished; it must wait before reading X.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <int M, bool DUAL>
__global__ void __launch_bounds__(GT, CTAS_PER_SM)
skinny_gemm_kernel(const GemmParams p) {
    constexpr int R = RowsPerWarp<M, DUAL>::value;
    constexpr int NT = DUAL ? 2 : 1;
    constexpr int NV = NT * R * M;               // sums one warp produces per row group
    extern __shared__ __align__(16) float smem[];
    float* xs = smem;                            // [M][KSP], each 256-step stored as [half][lane][4]
    float* ss = xs + (size_t)M * p.KSP;          // [64] sum of squares per row over this K slice
    float* red_all = ss + 64;                    // [GW][NV][33]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int ks = blockIdx.x % p.kslices;
    const int cta_in_slice = blockIdx.x / p.kslices, ctas_per_slice = gridDim.x / p.kslices;
    const int k0 = ks * p.KSP;
    const int kw = min(p.K, k0 + p.KSP) - k0;
    const int steps = (kw + KSTEP - 1) / KSTEP;
    const int gw = cta_in_slice * GW + warp, nw = ctas_per_slice * GW;
    float* red = red_all + (size_t)warp * NV * 33;

    // weight row pointers of a row group (rows past N are clamped: loaded, never stored)
    const __nv_bfloat16* wrow[NT][R];
    auto set_rows = [&](int g) {
#pragma unroll
        for (int rr = 0; rr < R; ++rr) {
            int n = g * R + rr;
            if (n >= p.N) n = p.N - 1;
            wrow[0][rr] = p.W + (size_t)n * p.K + k0 + lane * 8;
            if (DUAL) wrow[NT - 1][rr] = p.W2 + (size_t)n * p.K + k0 + lane * 8;
        }
    };
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
    uint4 wcur[NT][R], wnext[NT][R];
    int g = gw;
    if (g < p.groups) {                          // first loads go out before the dependency wait
        set_rows(g);
#pragma unroll
        for (int t = 0; t < NT; ++t)
#pragma unroll
            for (int rr = 0; rr < R; ++rr) wcur[t][rr] = (lane * 8 < kw) ? ldg_stream(wrow[t][rr]) : zero4;
    }
    grid_dependency_wait();
    grid_launch_dependents();

    // ---- stage the X slice (times the norm gain), permuted for conflict-free 128-bit reads:
    //      k = s*256 + lane*8 + h*4 + i  ->  s*256 + h*128 + lane*4 + i
    for (int idx = tid; idx < M * steps * (KSTEP / 4); idx += GT) {
        const int r = idx / (steps * (KSTEP / 4)), q4 = idx % (steps * (KSTEP / 4));
        const int kk = q4 * 4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (kk < kw) {                            // kw is a multiple of 8
            v = *reinterpret_cast<const float4*>(p.X + (size_t)r * p.ldx + k0 + kk);
            if (p.gain) {
                const uint2 gb = *reinterpret_cast<const uint2*>(p.gain + k0 + kk);
                v.x *= bf16lo(gb.x); v.y *= bf16hi(gb.x); v.z *= bf16lo(gb.y); v.w *= bf16hi(gb.y);
            }
        }
        const int s = kk >> 8, o = kk & 255;
        const int pos = (s << 8) + (((o >> 2) & 1) << 7) + ((o >> 3) << 2);
        *reinterpret_cast<float4*>(xs + (size_t)r * p.KSP + pos) = v;
    }
    if (p.gain) {
        for (int r = warp; r < M; r += GW) {
            float a = 0.f;
            for (int kk = lane * 4; kk < kw; kk += 128) {
                const float4 v = *reinterpret_cast<const float4*>(p.X + (size_t)r * p.ldx + k0 + kk);
                a = fmaf(v.x, v.x, a); a = fmaf(v.y, v.y, a); a = fmaf(v.z, v.z, a); a = fmaf(v.w, v.w, a);
            }
            a = warp_sum(a);
            if (lane == 0) ss[r] = a;
        }
    }
    __syncthreads();
    float* ss_part = p.partial + (size_t)p.kslices * p.groups * NV;   // [kslices][M]
    if (p.kslices > 1 && p.gain) {
        if (tid < M) ss_part[ks * M + tid] = ss[tid];
        __threadfence();
        __syncthreads();
    }

    for (; g < p.groups; g += nw) {
        float acc[NT][R][M];
#pragma unroll
        for (int t = 0; t < NT; ++t)
#pragma unroll
            for (int rr = 0; rr < R; ++rr)
#pragma unroll
                for (int r = 0; r < M; ++r) acc[t][rr][r] = 0.f;
        const int g_next = g + nw;
        for (int s = 0; s < steps; ++s) {
            // prefetch the next step, or the first step of this warp's next row group
            if (s + 1 < steps) {
                const bool ok = (s + 1) * KSTEP + lane * 8 < kw;
#pragma unroll
                for (int t = 0; t < NT; ++t)
#pragma unroll
                    for (int rr = 0; rr < R; ++rr)
                        wnext[t][rr] = ok ? ldg_stream(wrow[t][rr] + (s + 1) * KSTEP) : zero4;
            } else if (g_next < p.groups) {
                set_rows(g_next);
#pragma unroll
                for (int t = 0; t < NT; ++t)
#pragma unroll
                    for (int rr = 0; rr < R; ++rr) wnext[t][rr] = (lane * 8 < kw) ? ldg_stream(wrow[t][rr]) : zero4;
            }
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
        // ---- sum over lanes through shared memory: value v of lane l -> red[v][l]
        __syncwarp();
#pragma unroll
        for (int t = 0; t < NT; ++t)
#pragma unroll
            for (int rr = 0; rr < R; ++rr)
#pragma unroll
                for (int r = 0; r < M; ++r) red[((t * R + rr) * M + r) * 33 + lane] = acc[t][rr][r];
        __syncwarp();
        for (int v = lane; v < NV; v += 32) {
            const float* row = red + v * 33;
            float sum = 0.f;
#pragma unroll
            for (int j = 0; j < 32; ++j) sum += row[j];
            red[v * 33 + 32] = sum;              // column 32 holds the finished sum
        }
        __syncwarp();
        if (p.kslices > 1) {
            float* mine = p.partial + ((size_t)ks * p.groups + g) * NV;
            for (int v = lane; v < NV; v += 32) mine[v] = red[v * 33 + 32];
            __threadfence();
            __syncwarp();
            unsigned old = 0;
            if (lane == 0) old = atomicAdd(&p.tickets[g], 1u);
            old = __shfl_sync(0xffffffffu, old, 0);
            if (old != (unsigned)p.kslices - 1u) continue;     // another slice finishes this group
            __threadfence();
            for (int v = lane; v < NV; v += 32) {
                float sum = 0.f;
                for (int c = 0; c < p.kslices; ++c) sum += __ldcg(p.partial + ((size_t)c * p.groups + g) * NV + v);
                red[v * 33 + 32] = sum;
            }
            if (lane == 0) p.tickets[g] = 0u;                  // ready for the next launch
            __syncwarp();
        }
        // ---- epilogue: lane handles (row of the group, block row)
        for (int v = lane; v < R * M; v += 32) {
            const int rr = v / M, r = v % M, n = g * R + rr;
            if (n >= p.N) continue;
            float scale = 1.f;
            if (p.gain) {
                float q = ss[r];
                if (p.kslices > 1) {
                    q = 0.f;
                    for (int c = 0; c < p.kslices; ++c) q += __ldcg(ss_part + c * M + r);
                }
                scale = 1.f / sqrtf(q / (float)p.K + p.eps);
            }
            float val = red[v * 33 + 32] * scale;
            if (DUAL) {
                const float up = red[(R * M + v) * 33 + 32] * scale;
                val = (p.epilogue == EPI_GEGLU ? gelu_tanh_f(val) : silu_f(val)) * up;
            }
            float* y = p.Y + (size_t)r * p.ldy + n;
            if (p.epilogue == EPI_ADD) *y += val; else *y = val;
        }
        __syncwarp();
    }
}

template <int M, bool DUAL>
static csd_status launch_one(const GemmParams& gp, const LinearPlan& pl, cudaStream_t st) {
    auto kern = skinny_gemm_kernel<M, DUAL>;
    static bool attr_set = false;   // per instantiation
    if (!attr_set) {
        CSD_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BUDGET + 4096));
        attr_set = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)pl.grid);
    cfg.blockDim = dim3(GT);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    CSD_CUDA(cudaLaunchKernelEx(&cfg, kern, gp));
    count_launch();
    return CSD_OK;
}

size_t linear_scratch_bytes(int m, int N, int K, bool dual) {
    size_t worst = 0;
    for (int mm = 1; mm <= m; ++mm) {
        LinearPlan pl = plan_linear(mm, N, K, dual);
        size_t b = pl.scratch_floats * sizeof(float);
        if (b > worst) worst = b;
    }
    const size_t tc = tc_scratch_bytes(m, N, K, dual);
    if (tc > worst) worst = tc;
    return align_up(worst, 256);
}

int linear_ticket_count(int N) { return N + 1; }   // one ticket per row group, at least one row each

bool linear_uses_tensor_cores(int m, int N, int K, bool dual) {
    const int path = gemm_path();
    // measured on the 7B layer shapes the tensor-core kernel wins at every m (a 5-row review forward
    // takes 4.0 ms against 5.2 ms, a 17-row one 5.5 ms against 15 ms); tiny matrices stay on the simpler kernel
    return path != 1 && tc_supported(m, N, K, dual) && (path == 2 || (long long)N * K >= AUTO_TC_MIN_WEIGHTS);
}

// Which tensor-core kernel.  One tcgen05.mma reads 128 rows of shared memory for its wide operand
// and takes about 80 cycles whatever part of them is a CTA's own range, so the row-range kernel
// keeps up with the memory stream only where a range fills most of those rows.  Measured on the 7B
// shapes at 5 rows, each GEMM alone: 84 rows of the fused q|k|v projection 19 us against 20 with
// equal shares and a fix-up pass, 109 rows of the vocabulary projection equal, the 28 rows of the
// projections back to d_model 35 us against 17; inside a forward, where consecutive kernels overlap,
// the row-range kernel on q|k|v costs 5 us per layer more than it saves.  It is therefore chosen
// only on request (path 3) and stays as the comparison kernel without any cross-CTA traffic.
bool linear_uses_row_ranges(int m, int N, int K, bool dual) {
    if (!linear_uses_tensor_cores(m, N, K, dual) || !rs_supported(m, N, K, dual)) return false;
    return gemm_path() == 3;
}

int linear_ssq_pieces(int m, int N, int K, bool dual) {
    return linear_uses_row_ranges(m, N, K, dual) ? rs_ssq_pieces(m, N, K, dual) : 4 * ((N + 127) / 128);
}

int linear_ssq_capacity(int N) {
    const int sms = tc_sm_count(), per = (N + sms - 1) / sms, T = (per + 127) / 128;
    const int a = 4 * ((N + 127) / 128), b = sms * T * 4;
    return a > b ? a : b;
}

csd_status launch_linear(const LinearArgs& a, cudaStream_t st) {
    if (!a.W || !a.X || !a.Y || a.m < 1 || a.m > CSD_MAX_ROWS || a.N < 1 || a.K < 8 || (a.K & 7))
        return CSD_ERR_INVALID_ARG;
    const bool dual = a.W2 != nullptr;
    if (dual != (a.epilogue == EPI_SWIGLU || a.epilogue == EPI_GEGLU)) return CSD_ERR_INVALID_ARG;
    if ((((uintptr_t)a.W) & 15) || (dual && (((uintptr_t)a.W2) & 15))) return CSD_ERR_INVALID_ARG;
    if (a.xs && linear_uses_row_ranges(a.m, a.N, a.K, dual)) return launch_linear_rs(a, st);
    if (a.xs && linear_uses_tensor_cores(a.m, a.N, a.K, dual)) return launch_linear_tc(a, st);
    if ((((uintptr_t)a.X) & 15) || (a.ldx & 3)) return CSD_ERR_INVALID_ARG;
    const LinearPlan pl = plan_linear(a.m, a.N, a.K, dual);
    if (pl.kslices > 1 && (!a.partial || !a.tickets)) return CSD_ERR_INVALID_ARG;
    GemmParams gp;
    gp.W = a.W; gp.W2 = a.W2; gp.X = a.X; gp.gain = a.gain; gp.Y = a.Y; gp.partial = a.partial;
    gp.tickets = a.tickets; gp.N = a.N; gp.K = a.K; gp.ldx = a.ldx; gp.ldy = a.ldy; gp.m = a.m;
    gp.steps_per = pl.steps_per; gp.kslices = pl.kslices; gp.KSP = pl.KSP; gp.groups = pl.groups;
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

extern "C" csd_status csd_set_gemm_path(int path) {
    if (path < 0 || path > 3) return CSD_ERR_INVALID_ARG;
    set_gemm_path(path);
    return CSD_OK;
}

struct LinearWs { size_t tickets, partial, xs, ssq, total; };
static LinearWs linear_ws(int m, int N, int K) {
    LinearWs w;
    size_t off = 0;
    const int rows = m > CSD_MAX_ROWS ? CSD_WIDE_ROWS : CSD_MAX_ROWS;
    w.tickets = off; off += align_up((size_t)linear_ticket_count(N) * sizeof(unsigned), 256);
    w.partial = off;
    {
        size_t pb = linear_scratch_bytes(m > CSD_MAX_ROWS ? CSD_MAX_ROWS : m, N, K, false);
        if (m > CSD_MAX_ROWS && wide_partial_bytes(m, N, K, false) > pb) pb = wide_partial_bytes(m, N, K, false);
        off += pb;
    }
    w.xs = off;      off += align_up((size_t)3 * rows * K * 2, 256);
    w.ssq = off;     off += align_up((size_t)split_ssq_entries(K) * rows * sizeof(float), 256);
    w.total = off;
    return w;
}

extern "C" size_t csd_linear_workspace_bytes(int m, int N, int K) {
    if (m < 1 || m > CSD_WIDE_ROWS || N < 1 || K < 8) return 0;
    return linear_ws(m, N, K).total;
}

// The workspace must be zero before the first call (the ticket words live in it); every launch
// leaves the tickets zero again, so one cudaMemset after allocation is enough.
extern "C" csd_status csd_linear(const void* W_bf16_dev, int N, int K, const float* X_dev, int m, float* Y_dev,
                                 void* workspace_dev, size_t workspace_bytes, void* stream) {
    if (m < 1 || m > CSD_WIDE_ROWS || N < 1 || K < 8 || (K & 7)) return CSD_ERR_INVALID_ARG;
    if (!W_bf16_dev || !X_dev || !Y_dev || !workspace_dev) return CSD_ERR_INVALID_ARG;
    const LinearWs w = linear_ws(m, N, K);
    if (workspace_bytes < w.total) return CSD_ERR_CAPACITY;
    if (((uintptr_t)workspace_dev) & 255) return CSD_ERR_INVALID_ARG;
    char* ws = (char*)workspace_dev;
    if (m > CSD_MAX_ROWS) {                  // wide block: two-term rows, the wide tensor-core kernel
        if (!wide_supported(m, N, K, false)) return CSD_ERR_UNSUPPORTED;
        csd_status s = launch_wide_split(X_dev, K, K, m, nullptr, (__nv_bfloat16*)(ws + w.xs), nullptr, (cudaStream_t)stream);
        if (s != CSD_OK) return s;
        WideArgs wa;
        wa.W = (const __nv_bfloat16*)W_bf16_dev; wa.N = N; wa.K = K; wa.m = m; wa.xs = (const __nv_bfloat16*)(ws + w.xs);
        wa.Y = Y_dev; wa.ldy = N; wa.epilogue = EPI_STORE; wa.partial = (float*)(ws + w.partial);
        return launch_linear_wide(wa, (cudaStream_t)stream);
    }
    LinearArgs a;
    a.W = (const __nv_bfloat16*)W_bf16_dev; a.N = N; a.K = K; a.X = X_dev; a.ldx = K; a.m = m;
    a.Y = Y_dev; a.ldy = N; a.epilogue = EPI_STORE;
    a.tickets = (unsigned*)(ws + w.tickets);
    a.partial = (float*)(ws + w.partial);
    a.xs = (__nv_bfloat16*)(ws + w.xs);
    a.ssq = (float*)(ws + w.ssq);
    return launch_linear(a, (cudaStream_t)stream);
}
