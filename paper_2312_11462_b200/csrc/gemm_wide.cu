// Wide-block variant of the tensor-core GEMM  Y[m, N] = X[m, K] . W[N, K]^T  for up to 128 rows:
// the prompt prefill and the encoder pass, where the model takes many tokens in one run
// (Section 2) and the weights should stream once per 128 tokens instead of once per 17.
//
// Same plan as the row-range kernel (gemm_rs.cu): every CTA owns contiguous ranges of at most 128
// weight rows over the whole K extent, nothing is shared between CTAs.  The rows of X are the
// narrow operand of tcgen05.mma with up to 256 columns: each fp32 value enters as TWO bf16 terms
// x = hi + lo (16 mantissa bits, relative error 2^-17, the size of the tensor cores' own fp32
// accumulation error), laid out as [2][mpad][K] with mpad = m rounded up to 16, so one TMA box of
// 2*mpad rows brings both terms of a 64-wide K block.  With 128 rows a stage moves 32 KB of X for
// 11 to 16 KB of weights, all CTAs re-read X from L2, and the kernel is bound by what an SM can
// take in (about 63 GB/s), not by HBM; it still is one pass over the weights instead of eight.
// One CTA per SM (the ring takes most of the shared memory).
//
// Epilogue per output column (one thread per weight row): hi + lo sums, rms factor, residual add or
// gated activation, optional two-term split and sum-of-squares pieces for the next wide GEMM.
// Every mbarrier wait is bounded; on a time-out the CTA records CSD_ERR_TIMEOUT, stops, frees its
// tensor memory, returns.
#include "gemm_tc.cuh"
#include "tc_common.cuh"

namespace csd {

constexpr size_t WG_SMEM_MAX = 200 * 1024;
constexpr int WG_MAX_STAGES = 8;
constexpr int WG_THREADS = 320;              // TMA warp, MMA warp, eight epilogue warps (two per tensor-memory quadrant)

struct WgPlan {
    int mpad, npad, grid, T, V, box, rows8, ks, nkb, nks, stages, qp, chunks, tmem_cols, pk;
    size_t stage, smem;
};

struct __align__(8) WgCtrl {
    uint64_t full[WG_MAX_STAGES], empty[WG_MAX_STAGES], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    int abort_flag;
    float scale[CSD_WIDE_ROWS];
};

// K partitions: a matrix with few rows per CTA (the projections back to d_model) makes every CTA
// re-read all of X for a sliver of weights.  Cutting K in `pk` parts and the rows in grid / pk
// ranges of up to 128 divides the X traffic per CTA by pk; the pk partial results go to planes of
// a scratch buffer and a small kernel adds them (and runs the epilogue).  Only without an input
// norm, for single matrices with N a multiple of 8.
int wide_split_pieces(int K) { return (K + 1023) / 1024; }

int wide_pk(int m, int N, int K, bool dual) {
    (void)m;
    if (dual || (N & 7)) return 1;
    const int sms = tc_sm_count();
    if ((N + sms - 1) / sms >= 64 || K < 2048) return 1;
    int pk = sms / ((N + TILE_N - 1) / TILE_N);
    if (pk > 4) pk = 4;
    return pk < 2 ? 1 : pk;
}

static WgPlan wg_plan(int m, int N, int K, bool dual, int pk = 1) {
    WgPlan p{};
    p.mpad = (m + 15) & ~15;
    p.npad = 2 * p.mpad;
    p.pk = pk;
    p.grid = tc_sm_count();
    const int per = (N + p.grid - 1) / p.grid;
    p.T = (per + TILE_N - 1) / TILE_N;
    p.V = p.grid * p.T;
    if (pk > 1) { p.T = 1; p.V = p.grid / pk; p.grid = p.V * pk; }
    p.box = (N + p.V - 1) / p.V;
    p.rows8 = (p.box + 7) & ~7;
    p.qp = (p.box + 31) / 32;
    p.nkb = (K + KB - 1) / KB;
    const size_t wblk = (size_t)p.rows8 * 128, xb = (size_t)p.npad * 128;
    const size_t kblk = (dual ? 2 : 1) * wblk + xb;
    p.ks = kblk <= 24 * 1024 && p.nkb >= 2 ? 2 : 1;
    p.nks = (p.nkb + p.ks - 1) / p.ks;
    p.stage = (size_t)p.ks * kblk;
    // accumulator chunks of about 16 K blocks, as many as tensor memory holds (256 columns when the
    // accumulators fit them, all 512 otherwise), double-buffered when a CTA has two ranges
    const int acc_cols = p.npad * (dual ? 2 : 1), bufs = p.T > 1 ? 2 : 1;
    int chunks = (p.nkb + 15) / 16;
    const int room = (acc_cols * bufs <= 256 ? 256 : 512) / (acc_cols * bufs);
    if (chunks > room) chunks = room;
    if (chunks > p.nks / pk) chunks = p.nks / pk;
    p.chunks = chunks;                       // 0: the accumulators do not fit tensor memory
    p.tmem_cols = 32;
    while (p.tmem_cols < acc_cols * bufs * (chunks > 0 ? chunks : 1)) p.tmem_cols *= 2;
    const size_t reach = 16384 > wblk + xb ? 16384 - wblk - xb : 0;
    size_t tail = (sizeof(WgCtrl) + 127) & ~(size_t)127;
    if (tail < reach) tail = reach;
    p.stages = (int)((WG_SMEM_MAX - 1024 - tail) / p.stage);
    if (p.stages > WG_MAX_STAGES) p.stages = WG_MAX_STAGES;
    p.smem = (size_t)p.stages * p.stage + tail + 1024;
    return p;
}

bool wide_supported(int m, int N, int K, bool dual) {
    if (m < 1 || m > CSD_WIDE_ROWS || N < 1 || K < 64 || (K & 7)) return false;
    if ((long long)N * K < (1LL << 20)) return false;
    const WgPlan p = wg_plan(m, N, K, dual);
    return p.stages >= 2 && p.box >= 8 && p.chunks >= 1 && p.tmem_cols <= 512;
}

int wide_ssq_pieces(int m, int N, int K, bool dual) {
    if (wide_pk(m, N, K, dual) > 1) return wide_split_pieces(N);      // written by the kernel that adds the partial planes
    const WgPlan p = wg_plan(m, N, K, dual);
    return p.V * p.qp;
}
size_t wide_partial_bytes(int m, int N, int K, bool dual) {
    const int pk = wide_pk(m, N, K, dual);
    return pk > 1 ? align_up((size_t)pk * m * N * sizeof(float), 256) : 0;
}
int wide_ssq_capacity(int N) {
    const int sms = tc_sm_count(), per = (N + sms - 1) / sms, T = (per + 127) / 128;
    const int a = sms * T * 4, b = wide_split_pieces(N) + 1;     // GEMM epilogue pieces, split-kernel pieces
    return a > b ? a : b;
}

struct WgParams {
    float* Y; int* status;
    const float* ssq_in; int ssq_cnt;
    __nv_bfloat16* out_xs; const __nv_bfloat16* out_gain; float* out_ssq; int out_ld;
    int m, mpad, npad, N, K, ldy, nks, ks, T, V, box, rows8, stages, qp, chunks, tmem_cols, epilogue, pk;
    size_t plane;                       // floats between the partial planes of a K-partitioned launch
    float eps;
};

__device__ __forceinline__ float wg_gelu(float x) {
    return 0.5f * x * (1.f + tanhf(0.7978845608028654f * (x + 0.044715f * x * x * x)));
}
__device__ __forceinline__ float wg_silu(float x) { return x / (1.f + expf(-x)); }

// x = hi + lo with bf16 terms (16 mantissa bits)
__device__ __forceinline__ void split2f(float x, uint16_t& hi, uint16_t& lo) {
    hi = float_to_bf16_bits(x);
    lo = float_to_bf16_bits(x - bf16_bits_to_float(hi));
}

template <bool DUAL>
__global__ void __launch_bounds__(WG_THREADS, 1)
wide_gemm_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmW2,
                 const __grid_constant__ CUtensorMap tmX, const WgParams p) {
    constexpr int NT = DUAL ? 2 : 1;
    const int NPAD = p.npad, ACC_COLS = NPAD * NT;
    const uint32_t XBYTES = (uint32_t)NPAD * 128u;
    const uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NPAD >> 3) << 17) |
                           ((uint32_t)(TILE_N >> 4) << 24);   // f32 accumulate, bf16 x bf16, K-major both

    extern __shared__ unsigned char smem_raw[];
    unsigned char* ring = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t wblk = (uint32_t)p.rows8 * 128u;
    const uint32_t kblk = NT * wblk + XBYTES;                 // one K block of a stage: weights, then the rows' terms
    const uint32_t stage_bytes = (uint32_t)p.ks * kblk;
    WgCtrl* ctl = (WgCtrl*)(ring + (size_t)p.stages * stage_bytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int kslice = p.pk > 1 ? (int)blockIdx.x % p.pk : 0;       // this CTA's part of the K extent ...
    const int cta = p.pk > 1 ? (int)blockIdx.x / p.pk : (int)blockIdx.x;   // ... and its row ranges
    const int ks0 = kslice * p.nks / p.pk, nloc = (kslice + 1) * p.nks / p.pk - ks0;
    const int items = p.T * nloc;
    const int koff = (int)(((long long)blockIdx.x * nloc) / gridDim.x);   // every CTA starts at its own K stage
    const uint32_t tx_bytes = (uint32_t)p.ks * (NT * (uint32_t)p.box * 128u + XBYTES);

    if (tid == 0) {
        for (int s = 0; s < WG_MAX_STAGES; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&ctl->acc_full[b], 1); mbar_init(&ctl->acc_empty[b], 8); }
        ctl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&ctl->tmem_base)), "r"((uint32_t)p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctl->tmem_base;
    volatile int* abort_flag = &ctl->abort_flag;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == 0) {
        if (lane == 0) {
            struct Cursor { int t, j, kq, row0; };
            auto range_row = [&](int t) { return (int)(((long long)(cta * p.T + t) * p.N) / p.V); };
            auto step = [&](Cursor& c) {
                if (++c.kq == ks0 + nloc) c.kq = ks0;
                if (++c.j == nloc) { c.j = 0; ++c.t; c.row0 = range_row(c.t); }
            };
            auto load_w = [&](const Cursor& c, int s) {
                unsigned char* dst = ring + (size_t)s * stage_bytes;
                int x = c.kq * p.ks * KB;
                mbar_expect_tx(&ctl->full[s], tx_bytes);
                for (int h = 0; h < p.ks; ++h, x += KB, dst += kblk) {
                    tma_load_2d(dst, &tmW, &ctl->full[s], x, c.row0);
                    if (DUAL) tma_load_2d(dst + wblk, &tmW2, &ctl->full[s], x, c.row0);
                }
            };
            auto load_x = [&](const Cursor& c, int s) {
                unsigned char* dst = ring + (size_t)s * stage_bytes + NT * wblk;
                int x = c.kq * p.ks * KB;
                for (int h = 0; h < p.ks; ++h, x += KB, dst += kblk) tma_load_2d(dst, &tmX, &ctl->full[s], x, 0);
            };
            const int pre = items < p.stages ? items : p.stages;
            Cursor cw{0, 0, ks0 + koff, range_row(0)};
            Cursor cx = cw;
            for (int i = 0; i < pre; ++i) { load_w(cw, i); step(cw); }
            asm volatile("griddepcontrol.wait;" ::: "memory");
            for (int i = 0; i < pre; ++i) { load_x(cx, i); step(cx); }
            int s = 0;
            uint32_t ph = 0;
            for (int i = pre; i < items && !*abort_flag; ++i) {
                if (!mbar_wait(&ctl->empty[s], ph)) { *abort_flag = 1; break; }
                load_w(cw, s);
                load_x(cw, s);
                step(cw);
                if (++s == p.stages) { s = 0; ph ^= 1u; }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            const uint64_t desc0 = smem_desc_sw128(smem_u32(ring));
            for (int t = 0; t < p.T && !*abort_flag; ++t) {
                const int b = t & 1;
                if (!mbar_wait(&ctl->acc_empty[b], ((t >> 1) & 1) ^ 1)) { *abort_flag = 1; break; }
                tc_fence_after();
                uint32_t d0 = tmem + (uint32_t)(b * p.chunks * ACC_COLS);
                int rem = 0;
                bool fresh = true;
                for (int j = 0; j < nloc; ++j) {
                    if (!mbar_wait(&ctl->full[s], ph)) { *abort_flag = 1; break; }
                    tc_fence_after();
                    uint64_t ad = desc0 + (uint64_t)(((uint32_t)s * stage_bytes) >> 4);
                    for (int h = 0; h < p.ks; ++h, ad += kblk >> 4) {
                        const uint64_t bd = ad + ((NT * wblk) >> 4);
#pragma unroll
                        for (int k = 0; k < KB / 16; ++k) {
                            const uint32_t acc = (fresh && (h | k) == 0) ? 0u : 1u;
                            tc_mma(d0, ad + 2 * k, bd + 2 * k, IDESC, acc);
                            if (DUAL) tc_mma(d0 + NPAD, ad + (wblk >> 4) + 2 * k, bd + 2 * k, IDESC, acc);
                        }
                    }
                    tc_commit(&ctl->empty[s]);
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                    rem += p.chunks;
                    fresh = rem >= nloc;
                    if (fresh) { rem -= nloc; d0 += ACC_COLS; }
                }
                if (*abort_flag) break;
                tc_commit(&ctl->acc_full[b]);
            }
        }
    } else {
        // ---- epilogue warps: quadrant q of tensor memory holds weight rows q*32 .. q*32+31 of the range;
        //      the two warps of a quadrant take the 16-row chunks of the block in turn
        const int q = warp & 3, ew = warp - 2, half = ew >> 2, m = p.m, mpad = p.mpad;
        asm volatile("griddepcontrol.wait;" ::: "memory");
        for (int r = ew; r < m; r += 8) {
            float sc = 1.f;
            if (p.ssq_in) {
                float sq = 0.f;
                for (int c = lane; c < p.ssq_cnt; c += 32) sq += __ldcg(p.ssq_in + (size_t)c * m + r);
                sq = warp_sum(sq);
                sc = 1.f / sqrtf(sq / (float)p.K + p.eps);
            }
            if (lane == 0) ctl->scale[r] = sc;
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        for (int t = 0; t < p.T; ++t) {
            const int b = t & 1, v = cta * p.T + t;
            const int row0 = (int)(((long long)v * p.N) / p.V), row1 = (int)(((long long)(v + 1) * p.N) / p.V);
            const int n = row0 + q * 32 + lane;
            const bool mine = n < row1;
            float out_g = 1.f;
            if (mine && p.out_xs && p.out_gain) out_g = __bfloat162float(p.out_gain[n]);
            if (!mbar_wait(&ctl->acc_full[b], (t >> 1) & 1)) { *abort_flag = 1; break; }
            tc_fence_after();
            const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * p.chunks * ACC_COLS);
            const int nchunk = (m + 15) / 16, my_last = ((nchunk - 1 - half) / 2) * 2 + half;   // this warp's last chunk
            if (half >= nchunk) {                // nothing to read: release the accumulators at once
                if (lane == 0) mbar_arrive(&ctl->acc_empty[b]);
                continue;
            }
            for (int r0 = 16 * half; r0 < m; r0 += 32) {
                float val[16], up[16], lo[16], lo2[16], yold[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) { val[i] = 0.f; up[i] = 0.f; lo[i] = 0.f; lo2[i] = 0.f; yold[i] = 0.f; }
                if (p.epilogue == EPI_ADD && mine) {   // the residual rows of this chunk, all requested at once
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (r0 + i < m) yold[i] = __ldcg(p.Y + (size_t)kslice * p.plane + (size_t)(r0 + i) * p.ldy + n);
                }
                for (int ch = 0; ch < p.chunks; ++ch) {
                    float a[16];
                    tc_ld16(taddr + (uint32_t)(ch * ACC_COLS + r0), a);
#pragma unroll
                    for (int i = 0; i < 16; ++i) val[i] += a[i];
                    tc_ld16(taddr + (uint32_t)(ch * ACC_COLS + mpad + r0), a);
#pragma unroll
                    for (int i = 0; i < 16; ++i) lo[i] += a[i];
                    if (DUAL) {
                        tc_ld16(taddr + (uint32_t)(ch * ACC_COLS + NPAD + r0), a);
#pragma unroll
                        for (int i = 0; i < 16; ++i) up[i] += a[i];
                        tc_ld16(taddr + (uint32_t)(ch * ACC_COLS + NPAD + mpad + r0), a);
#pragma unroll
                        for (int i = 0; i < 16; ++i) lo2[i] += a[i];
                    }
                }
                if (r0 == 16 * my_last) {         // this warp's last read of the accumulator set
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ctl->acc_empty[b]);
                }
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int r = r0 + i;
                    if (r < m) {                  // (uniform across the warp)
                        const float scale = ctl->scale[r];
                        float x = (val[i] + lo[i]) * scale;
                        if (DUAL) {
                            const float u = (up[i] + lo2[i]) * scale;
                            x = (p.epilogue == EPI_GEGLU ? wg_gelu(x) : wg_silu(x)) * u;
                        }
                        if (mine) {
                            float* y = p.Y + (size_t)kslice * p.plane + (size_t)r * p.ldy + n;
                            x += yold[i];
                            *y = x;
                        } else {
                            x = 0.f;              // lanes past the range carry garbage
                        }
                        if (p.out_ssq && q < p.qp) {
                            const float sq = warp_sum(x * x);
                            if (lane == 0) p.out_ssq[(size_t)(v * p.qp + q) * m + r] = sq;
                        }
                        if (p.out_xs && mine) {
                            uint16_t h1, l1;
                            split2f(x * out_g, h1, l1);
                            uint16_t* o = reinterpret_cast<uint16_t*>(p.out_xs) + n;
                            o[(size_t)r * p.out_ld] = h1;
                            o[(size_t)(mpad + r) * p.out_ld] = l1;
                        }
                    }
                }
            }
        }
    }
    if (*abort_flag) {
        if (tid == 0) set_status(p.status, CSD_ERR_TIMEOUT);
        __nanosleep(2000000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)p.tmem_cols) : "memory");
    }
}

// fp32 rows (times an optional gain) -> two bf16 terms [2][mpad][K] (rows m..mpad-1 zero), plus the
// pieces of each row's sum of squares.  grid = (K / 1024 rounded up, mpad).
__global__ void __launch_bounds__(128)
split2_rows_kernel(const float* __restrict__ X, int ldx, int K, int m, int mpad, const __nv_bfloat16* __restrict__ gain,
                   __nv_bfloat16* __restrict__ xs, float* __restrict__ ssq) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int r = blockIdx.y, k = (blockIdx.x * 128 + threadIdx.x) * 8;
    float sq = 0.f;
    if (k < K) {
        float v[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (r < m) {
            const float* src = X + (size_t)r * ldx + k;
            const float4 a = *reinterpret_cast<const float4*>(src), b = *reinterpret_cast<const float4*>(src + 4);
            v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) sq = fmaf(v[e], v[e], sq);
        if (gain) {
            const uint4 g = *reinterpret_cast<const uint4*>(gain + k);
            v[0] *= bf16lo(g.x); v[1] *= bf16hi(g.x); v[2] *= bf16lo(g.y); v[3] *= bf16hi(g.y);
            v[4] *= bf16lo(g.z); v[5] *= bf16hi(g.z); v[6] *= bf16lo(g.w); v[7] *= bf16hi(g.w);
        }
        uint32_t t[2][4];
#pragma unroll
        for (int e = 0; e < 8; e += 2) {
            uint16_t a1, a2, c1, c2;
            split2f(v[e], a1, a2);
            split2f(v[e + 1], c1, c2);
            t[0][e / 2] = a1 | ((uint32_t)c1 << 16); t[1][e / 2] = a2 | ((uint32_t)c2 << 16);
        }
#pragma unroll
        for (int s = 0; s < 2; ++s)
            *reinterpret_cast<uint4*>(xs + (size_t)(s * mpad + r) * K + k) = make_uint4(t[s][0], t[s][1], t[s][2], t[s][3]);
    }
    __shared__ float part[4];
    sq = warp_sum(sq);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = sq;
    __syncthreads();
    if (threadIdx.x == 0 && ssq && r < m) ssq[(size_t)blockIdx.x * m + r] = (part[0] + part[1]) + (part[2] + part[3]);
}

// Adds the partial planes of a K-partitioned launch in plane order, then the epilogue: optional
// residual add into Y, optional two-term split (times a gain) and sum-of-squares pieces.
// grid = (N / 1024 rounded up, m); N a multiple of 8.
__global__ void __launch_bounds__(128)
wide_reduce_kernel(const float* __restrict__ P, int pk, size_t plane, int N, int m, int mpad, float* __restrict__ Y, int ldy,
                   int add, const __nv_bfloat16* __restrict__ gain, __nv_bfloat16* __restrict__ xs, int out_ld,
                   float* __restrict__ ssq) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int r = blockIdx.y, k = (blockIdx.x * 128 + threadIdx.x) * 8;
    float sq = 0.f;
    if (k < N) {
        float v[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int j = 0; j < pk; ++j) {
            const float* src = P + (size_t)j * plane + (size_t)r * N + k;
            const float4 a = __ldcg(reinterpret_cast<const float4*>(src)), b = __ldcg(reinterpret_cast<const float4*>(src + 4));
            v[0] += a.x; v[1] += a.y; v[2] += a.z; v[3] += a.w; v[4] += b.x; v[5] += b.y; v[6] += b.z; v[7] += b.w;
        }
        float* y = Y + (size_t)r * ldy + k;
        if (add) {
            const float4 a = *reinterpret_cast<const float4*>(y), b = *reinterpret_cast<const float4*>(y + 4);
            v[0] += a.x; v[1] += a.y; v[2] += a.z; v[3] += a.w; v[4] += b.x; v[5] += b.y; v[6] += b.z; v[7] += b.w;
        }
        *reinterpret_cast<float4*>(y) = make_float4(v[0], v[1], v[2], v[3]);
        *reinterpret_cast<float4*>(y + 4) = make_float4(v[4], v[5], v[6], v[7]);
#pragma unroll
        for (int e = 0; e < 8; ++e) sq = fmaf(v[e], v[e], sq);
        if (xs) {
            if (gain) {
                const uint4 g = *reinterpret_cast<const uint4*>(gain + k);
                v[0] *= bf16lo(g.x); v[1] *= bf16hi(g.x); v[2] *= bf16lo(g.y); v[3] *= bf16hi(g.y);
                v[4] *= bf16lo(g.z); v[5] *= bf16hi(g.z); v[6] *= bf16lo(g.w); v[7] *= bf16hi(g.w);
            }
            uint32_t t[2][4];
#pragma unroll
            for (int e = 0; e < 8; e += 2) {
                uint16_t a1, a2, c1, c2;
                split2f(v[e], a1, a2);
                split2f(v[e + 1], c1, c2);
                t[0][e / 2] = a1 | ((uint32_t)c1 << 16); t[1][e / 2] = a2 | ((uint32_t)c2 << 16);
            }
#pragma unroll
            for (int s = 0; s < 2; ++s)
                *reinterpret_cast<uint4*>(xs + (size_t)(s * mpad + r) * out_ld + k) = make_uint4(t[s][0], t[s][1], t[s][2], t[s][3]);
        }
    }
    __shared__ float part[4];
    sq = warp_sum(sq);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = sq;
    __syncthreads();
    if (threadIdx.x == 0 && ssq) ssq[(size_t)blockIdx.x * m + r] = (part[0] + part[1]) + (part[2] + part[3]);
}

csd_status launch_wide_split(const float* X, int ldx, int K, int m, const __nv_bfloat16* gain, __nv_bfloat16* xs,
                             float* ssq, cudaStream_t st) {
    if (!X || !xs || (((uintptr_t)X) & 15) || (ldx & 3) || (K & 7) || m < 1 || m > CSD_WIDE_ROWS) return CSD_ERR_INVALID_ARG;
    const int mpad = (m + 15) & ~15;
    PdlLaunch L(dim3((unsigned)wide_split_pieces(K), (unsigned)mpad), dim3(128), 0, st);
    CSD_CUDA(cudaLaunchKernelEx(&L.cfg, split2_rows_kernel, X, ldx, K, m, mpad, gain, xs, ssq));
    count_launch();
    return CSD_OK;
}

template <bool DUAL>
static csd_status launch_wg(const CUtensorMap& tw, const CUtensorMap& tw2, const CUtensorMap& tx, const WgParams& wp,
                            const WgPlan& pl, cudaStream_t st) {
    auto kern = wide_gemm_kernel<DUAL>;
    static bool attr_set = false;
    if (!attr_set) {
        CSD_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)WG_SMEM_MAX));
        attr_set = true;
    }
    PdlLaunch L(dim3((unsigned)pl.grid), dim3(WG_THREADS), pl.smem, st);
    CSD_CUDA(cudaLaunchKernelEx(&L.cfg, kern, tw, tw2, tx, wp));
    count_launch();
    return CSD_OK;
}

csd_status launch_linear_wide(const WideArgs& a, cudaStream_t st) {
    const bool dual = a.W2 != nullptr;
    if (!a.W || !a.Y || !a.xs || (((uintptr_t)a.xs) & 15)) return CSD_ERR_INVALID_ARG;
    if (dual != (a.epilogue == EPI_SWIGLU || a.epilogue == EPI_GEGLU)) return CSD_ERR_INVALID_ARG;
    if (!wide_supported(a.m, a.N, a.K, dual)) return CSD_ERR_UNSUPPORTED;
    int pk = a.ssq ? 1 : wide_pk(a.m, a.N, a.K, dual);
    if (pk > 1 && (!a.partial || (a.ldy & 3) || (((uintptr_t)a.Y) & 15) || (a.out_xs && (a.out_ld & 7)))) return CSD_ERR_INVALID_ARG;
    const WgPlan pl = wg_plan(a.m, a.N, a.K, dual, pk);
    if (pk > 1 && (pl.box > TILE_N || pl.chunks < 1 || pl.stages < 2)) return CSD_ERR_UNSUPPORTED;
    CUtensorMap tw, tw2, tx;
    if (!tensor_map_2d(a.W, a.N, a.K, pl.box, &tw)) return CSD_ERR_UNSUPPORTED;
    tw2 = tw;
    if (dual && !tensor_map_2d(a.W2, a.N, a.K, pl.box, &tw2)) return CSD_ERR_UNSUPPORTED;
    if (!tensor_map_2d(a.xs, pl.npad, a.K, pl.npad, &tx)) return CSD_ERR_UNSUPPORTED;
    WgParams wp;
    wp.Y = a.Y; wp.status = status_word_device();
    wp.ssq_in = a.ssq; wp.ssq_cnt = a.ssq_cnt;
    wp.out_xs = a.out_xs; wp.out_gain = a.out_gain; wp.out_ssq = a.out_ssq; wp.out_ld = a.out_ld;
    wp.m = a.m; wp.mpad = pl.mpad; wp.npad = pl.npad; wp.N = a.N; wp.K = a.K; wp.ldy = a.ldy; wp.nks = pl.nks; wp.ks = pl.ks;
    wp.T = pl.T; wp.V = pl.V; wp.box = pl.box; wp.rows8 = pl.rows8; wp.stages = pl.stages; wp.qp = pl.qp;
    wp.chunks = pl.chunks; wp.tmem_cols = pl.tmem_cols; wp.epilogue = a.epilogue; wp.eps = a.eps;
    wp.pk = pk; wp.plane = 0;
    if (pk > 1) {                        // partial planes now, sums and epilogue in the small kernel after
        wp.Y = a.partial; wp.ldy = a.N; wp.plane = (size_t)a.m * a.N; wp.epilogue = EPI_STORE;
        wp.out_xs = nullptr; wp.out_ssq = nullptr; wp.out_gain = nullptr;
        const csd_status s = launch_wg<false>(tw, tw2, tx, wp, pl, st);
        if (s != CSD_OK) return s;
        PdlLaunch L(dim3((unsigned)wide_split_pieces(a.N), (unsigned)a.m), dim3(128), 0, st);
        CSD_CUDA(cudaLaunchKernelEx(&L.cfg, wide_reduce_kernel, (const float*)a.partial, pk, wp.plane, a.N, a.m, pl.mpad, a.Y,
                                    a.ldy, a.epilogue == EPI_ADD ? 1 : 0, a.out_gain, a.out_xs, a.out_ld, a.out_ssq));
        count_launch();
        return CSD_OK;
    }
    return dual ? launch_wg<true>(tw, tw2, tx, wp, pl, st) : launch_wg<false>(tw, tw2, tx, wp, pl, st);
}

}  // namespace csd
