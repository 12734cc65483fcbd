// Row-range variant of the tensor-core weight-streaming GEMM  Y[m, N] = X[m, K] . W[N, K]^T.
//
// The N weight rows (output columns) are cut into V = grid x T contiguous ranges of at most 128
// rows, range v = [v*N/V, (v+1)*N/V), and every CTA (one per SM) owns T consecutive ranges over the
// WHOLE K extent.  Nothing is shared between CTAs: no partial sums leave the chip, no ticket, no
// finishing pass; the tail of the kernel is one accumulator read and the stores.  All CTAs stream
// the same number of weight bytes to within one row.
//
// A range's rows are the 128-row operand of tcgen05.mma.  The TMA box is as high as the longest
// range; the instruction still reads 128 rows of shared memory from the box's start, so the lanes
// past the range hold products of whatever lies behind the box (the rows' terms, the next stage):
// finite or not, they stay in their own accumulator lanes and are never read.  The block's rows
// arrive as three bf16 terms per value (see gemm_tc.cu) and are the narrow operand; their 64-wide K
// block rides in the same stage as the weights' one.  A stage carries one to four K blocks so that
// one barrier round trip moves 20 to 32 KB.
//
// The tensor cores add into an fp32 accumulator with less care than an fp32 FMA chain, and the
// loss grows with the length of the chain, so the K extent is cut into chunks of about 1024
// elements, each with its own accumulator columns in tensor memory; the epilogue adds the chunks
// in fp32.
//
// Roles (192 threads): warp 0 lane 0 issues TMA, warp 1 lane 0 issues MMA, warps 2-5 read their
// quadrant of tensor memory and run the epilogue (rms factor, residual add or gated activation,
// optional three-term split and sum-of-squares pieces for the next GEMM).  The first ring-full of
// weight boxes is requested before the programmatic-dependent-launch wait.  Every mbarrier wait is
// bounded; on a time-out the CTA records CSD_ERR_TIMEOUT, stops, frees its tensor memory, returns.
#include "gemm_tc.cuh"
#include "tc_common.cuh"

namespace csd {

constexpr size_t RS_SMEM_MAX = 111 * 1024;              // two CTAs (of consecutive kernels) fit one SM
constexpr int RS_MAX_STAGES = 12;

static int rs_npad(int m) { int c = 3 * m; return c <= 16 ? 16 : (c <= 32 ? 32 : (c <= 48 ? 48 : 64)); }

struct RsPlan {
    int npad, grid, T, V, box, rows8, ks, nkb, nks, stages, qp, chunks, tmem_cols;
    size_t stage, smem;
};

struct __align__(8) RsCtrl {
    uint64_t full[RS_MAX_STAGES], empty[RS_MAX_STAGES], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    int abort_flag;
    float scale[32];
};

static RsPlan rs_plan(int m, int N, int K, bool dual) {
    RsPlan p{};
    p.npad = rs_npad(m);
    p.grid = tc_sm_count();
    const int per = (N + p.grid - 1) / p.grid;
    p.T = (per + TILE_N - 1) / TILE_N;
    p.V = p.grid * p.T;
    p.box = (N + p.V - 1) / p.V;
    p.rows8 = (p.box + 7) & ~7;
    p.qp = (p.box + 31) / 32;
    p.nkb = (K + KB - 1) / KB;
    const size_t wblk = (size_t)p.rows8 * 128, xb = (size_t)p.npad * 128;
    const size_t kblk = (dual ? 2 : 1) * wblk + xb;
    int ks = (int)((28 * 1024 + kblk / 2) / kblk);
    if (ks < 1) ks = 1;
    if (ks > 4) ks = 4;
    if (ks > p.nkb) ks = p.nkb;
    p.ks = ks;
    p.nks = (p.nkb + ks - 1) / ks;
    p.stage = (size_t)ks * kblk;
    // accumulator chunks: about 16 K blocks each, as many as fit 256 tensor-memory columns (the
    // next kernel's CTA on the same SM needs the other 256), double-buffered when a CTA has two ranges
    const int acc_cols = p.npad * (dual ? 2 : 1), bufs = p.T > 1 ? 2 : 1;
    int chunks = (p.nkb + 15) / 16;
    if (chunks > 256 / (acc_cols * bufs)) chunks = 256 / (acc_cols * bufs);
    if (chunks > p.nks) chunks = p.nks;
    if (chunks < 1) chunks = 1;
    p.chunks = chunks;
    p.tmem_cols = 32;
    while (p.tmem_cols < acc_cols * bufs * chunks) p.tmem_cols *= 2;
    // the last weight block of the ring is read 128 rows deep: what that reaches past the ring
    // must still lie inside this CTA's allocation
    const size_t reach = 16384 > wblk + xb ? 16384 - wblk - xb : 0;
    size_t tail = (sizeof(RsCtrl) + 127) & ~(size_t)127;
    if (tail < reach) tail = reach;
    p.stages = (int)((RS_SMEM_MAX - 1024 - tail) / p.stage);
    if (p.stages > RS_MAX_STAGES) p.stages = RS_MAX_STAGES;
    p.smem = (size_t)p.stages * p.stage + tail + 1024;
    return p;
}

bool rs_supported(int m, int N, int K, bool dual) {
    if (!tc_supported(m, N, K, dual)) return false;
    const RsPlan p = rs_plan(m, N, K, dual);
    return p.stages >= 2 && p.box >= 8;
}

int rs_ssq_pieces(int m, int N, int K, bool dual) {
    const RsPlan p = rs_plan(m, N, K, dual);
    return p.V * p.qp;
}

int rs_box_rows(int m, int N, int K, bool dual) { return rs_plan(m, N, K, dual).box; }

struct RsParams {
    float* Y; int* status;
    const float* ssq_in; int ssq_cnt;
    __nv_bfloat16* out_xs; const __nv_bfloat16* out_gain; float* out_ssq; int out_ld;
    int N, K, ldy, nks, ks, T, V, box, rows8, stages, qp, chunks, tmem_cols, epilogue;
    float eps;
};

__device__ __forceinline__ float rs_gelu(float x) {
    return 0.5f * x * (1.f + tanhf(0.7978845608028654f * (x + 0.044715f * x * x * x)));
}
__device__ __forceinline__ float rs_silu(float x) { return x / (1.f + expf(-x)); }

template <int M, bool DUAL>
__global__ void __launch_bounds__(TC_THREADS, 2)
skinny_gemm_rs_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmW2,
                      const __grid_constant__ CUtensorMap tmX, const RsParams p) {
    constexpr int NPAD = 3 * M <= 16 ? 16 : (3 * M <= 32 ? 32 : (3 * M <= 48 ? 48 : 64));
    constexpr int NT = DUAL ? 2 : 1;
    constexpr int ACC_COLS = NPAD * NT;                       // tensor-memory columns per accumulator set
    constexpr int XBYTES = NPAD * 128;                        // the rows' terms for one K block
    constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NPAD >> 3) << 17) |
                               ((uint32_t)(TILE_N >> 4) << 24);   // f32 accumulate, bf16 x bf16, K-major both

    extern __shared__ unsigned char smem_raw[];
    unsigned char* ring = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t wblk = (uint32_t)p.rows8 * 128u;           // one weight block: rows8 x 64 bf16
    const uint32_t kblk = NT * wblk + XBYTES;                 // one K block of a stage: weights, then the rows' terms
    const uint32_t stage_bytes = (uint32_t)p.ks * kblk;
    RsCtrl* ctl = (RsCtrl*)(ring + (size_t)p.stages * stage_bytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x;
    const int items = p.T * p.nks;                            // stages of work of this CTA
    // every CTA walks the K extent from its own starting stage (and wraps around): at any moment the
    // CTAs read different columns of the weights and different pieces of the rows' terms, which
    // spreads the requests over the memory channels and the L2 slices
    const int koff = (int)(((long long)cta * p.nks) / gridDim.x);
    const uint32_t tx_bytes = (uint32_t)p.ks * (NT * (uint32_t)p.box * 128u + XBYTES);

    if (tid == 0) {
        for (int s = 0; s < RS_MAX_STAGES; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&ctl->acc_full[b], 1); mbar_init(&ctl->acc_empty[b], 4); }
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
    // the next kernel in the stream may start now: it takes the second slot of each SM, sets up and
    // requests its first weight boxes; it touches nothing this kernel writes before its own wait
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == 0) {
        if (lane == 0) {
            // One thread walks the CTA's stages; all its index arithmetic is incremental (a division
            // here costs more than the copy instructions it feeds).
            struct Cursor {
                int t, j, kq, row0;               // range, stage inside it, rotated K stage, the range's first row
            };
            auto range_row = [&](int t) { return (int)(((long long)(cta * p.T + t) * p.N) / p.V); };
            auto step = [&](Cursor& c) {
                if (++c.kq == p.nks) c.kq = 0;
                if (++c.j == p.nks) { c.j = 0; ++c.t; c.row0 = range_row(c.t); }
            };
            auto load_w = [&](const Cursor& c, int s) {
                unsigned char* dst = ring + (size_t)s * stage_bytes;
                int x = c.kq * p.ks * KB;
                mbar_expect_tx(&ctl->full[s], tx_bytes);
                for (int h = 0; h < p.ks; ++h, x += KB, dst += kblk) {   // K blocks past K: the box is filled with zeros
                    tma_load_2d(dst, &tmW, &ctl->full[s], x, c.row0);
                    if (DUAL) tma_load_2d(dst + wblk, &tmW2, &ctl->full[s], x, c.row0);
                }
            };
            auto load_x = [&](const Cursor& c, int s) {
                unsigned char* dst = ring + (size_t)s * stage_bytes + NT * wblk;
                int x = c.kq * p.ks * KB;
                for (int h = 0; h < p.ks; ++h, x += KB, dst += kblk) tma_load_2d(dst, &tmX, &ctl->full[s], x, 0);
            };
            // the weights do not depend on the kernel that produces the rows: the first ring-full
            // goes out before the dependency wait, the rows' terms after it
            const int pre = items < p.stages ? items : p.stages;
            Cursor cw{0, 0, koff, range_row(0)};
            Cursor cx = cw;
            for (int i = 0; i < pre; ++i) { load_w(cw, i); step(cw); }
            asm volatile("griddepcontrol.wait;" ::: "memory");
            for (int i = 0; i < pre; ++i) { load_x(cx, i); step(cx); }
            int s = 0;
            uint32_t ph = 0;                      // parity of the phase of empty[s] that frees slot s next
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
            uint32_t ph = 0;                      // parity of the phase of full[s] that fills slot s next
            const uint64_t desc0 = smem_desc_sw128(smem_u32(ring));   // descriptors differ in the address field only
            for (int t = 0; t < p.T && !*abort_flag; ++t) {
                const int b = t & 1;
                if (!mbar_wait(&ctl->acc_empty[b], ((t >> 1) & 1) ^ 1)) { *abort_flag = 1; break; }
                tc_fence_after();
                uint32_t d0 = tmem + (uint32_t)(b * p.chunks * ACC_COLS);
                int rem = 0;                      // stage j adds into chunk floor(j * chunks / nks)
                bool fresh = true;
                for (int j = 0; j < p.nks; ++j) {
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
                    tc_commit(&ctl->empty[s]);          // stage reusable once these MMAs have read it
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                    rem += p.chunks;
                    fresh = rem >= p.nks;
                    if (fresh) { rem -= p.nks; d0 += ACC_COLS; }
                }
                if (*abort_flag) break;
                tc_commit(&ctl->acc_full[b]);           // this range's accumulators are complete
            }
        }
    } else {
        // ---- epilogue warps: quadrant q of tensor memory holds weight rows q*32 .. q*32+31 of the range
        const int q = warp & 3, ew = warp - 2;
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (p.ssq_in) {                         // rms factor of every row from the pieces of its sum of squares
            for (int r = ew; r < M; r += 4) {
                float sq = 0.f;
                for (int c = lane; c < p.ssq_cnt; c += 32) sq += __ldcg(p.ssq_in + (size_t)c * M + r);
                sq = warp_sum(sq);
                if (lane == 0) ctl->scale[r] = 1.f / sqrtf(sq / (float)p.K + p.eps);
            }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        for (int t = 0; t < p.T; ++t) {
            const int b = t & 1, v = cta * p.T + t;
            const int row0 = (int)(((long long)v * p.N) / p.V), row1 = (int)(((long long)(v + 1) * p.N) / p.V);
            const int row = q * 32 + lane, n = row0 + row;
            const bool mine = n < row1;
            // what the finishing step needs besides the sums travels while the MMAs run
            float yold[M];
            float out_g = 1.f;
#pragma unroll
            for (int r = 0; r < M; ++r) yold[r] = 0.f;
            if (mine) {
                if (p.epilogue == EPI_ADD) {
#pragma unroll
                    for (int r = 0; r < M; ++r) yold[r] = __ldcg(p.Y + (size_t)r * p.ldy + n);
                }
                if (p.out_xs && p.out_gain) out_g = __bfloat162float(p.out_gain[n]);
            }
            if (!mbar_wait(&ctl->acc_full[b], (t >> 1) & 1)) { *abort_flag = 1; break; }   // same outcome in all four warps
            tc_fence_after();
            const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * p.chunks * ACC_COLS);
            float sums[NT][M];
#pragma unroll
            for (int u = 0; u < NT; ++u) {
                float third[M], second[M];
#pragma unroll
                for (int r = 0; r < M; ++r) { sums[u][r] = 0.f; second[r] = 0.f; third[r] = 0.f; }
                for (int ch = 0; ch < p.chunks; ++ch) {       // chunks of the K extent, in order
#pragma unroll
                    for (int c0 = 0; c0 < NPAD; c0 += 16) {
                        if (c0 >= 3 * M) break;
                        float vv[16];
                        tc_ld16(taddr + (uint32_t)(ch * ACC_COLS + u * NPAD + c0), vv);
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            const int col = c0 + c;
                            if (col < M) sums[u][col] += vv[c];
                            else if (col < 2 * M) second[col - M] += vv[c];
                            else if (col < 3 * M) third[col - 2 * M] += vv[c];
                        }
                    }
                }
#pragma unroll
                for (int r = 0; r < M; ++r) sums[u][r] += second[r] + third[r];   // small terms first
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->acc_empty[b]);
            float outv[M];
#pragma unroll
            for (int r = 0; r < M; ++r) {
                const float scale = p.ssq_in ? ctl->scale[r] : 1.f;
                float val = sums[0][r] * scale;
                if (DUAL) {
                    const float up = sums[NT - 1][r] * scale;
                    val = (p.epilogue == EPI_GEGLU ? rs_gelu(val) : rs_silu(val)) * up;
                }
                if (mine) {
                    if (p.epilogue == EPI_ADD) val += yold[r];
                    p.Y[(size_t)r * p.ldy + n] = val;
                } else {
                    val = 0.f;                          // lanes past the range carry garbage
                }
                outv[r] = val;
            }
            if (p.out_ssq && q < p.qp) {          // pieces of the rows' sums of squares, one per 32 columns
#pragma unroll
                for (int r = 0; r < M; ++r) {
                    const float sq = warp_sum(outv[r] * outv[r]);
                    if (lane == 0) p.out_ssq[(size_t)(v * p.qp + q) * M + r] = sq;
                }
            }
            if (p.out_xs && mine) {               // the rows as three bf16 terms for the GEMM that reads them next
#pragma unroll
                for (int r = 0; r < M; ++r) {
                    uint16_t b1, b2, b3;
                    split3(outv[r] * out_g, b1, b2, b3);
                    uint16_t* o = reinterpret_cast<uint16_t*>(p.out_xs) + n;
                    o[(size_t)r * p.out_ld] = b1;
                    o[(size_t)(M + r) * p.out_ld] = b2;
                    o[(size_t)(2 * M + r) * p.out_ld] = b3;
                }
            }
        }
    }
    if (*abort_flag) {
        if (tid == 0) set_status(p.status, CSD_ERR_TIMEOUT);
        __nanosleep(2000000);          // let copies already in flight land before the CTA's memory is released
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)p.tmem_cols) : "memory");
    }
}

template <int M, bool DUAL>
static csd_status launch_rs(const CUtensorMap& tw, const CUtensorMap& tw2, const CUtensorMap& tx, const RsParams& rp,
                            const RsPlan& pl, cudaStream_t st) {
    auto kern = skinny_gemm_rs_kernel<M, DUAL>;
    static bool attr_set = false;
    if (!attr_set) {
        CSD_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)RS_SMEM_MAX));
        // ask for the largest shared-memory carve-out, or the second CTA (the next kernel's) does not fit
        CSD_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
        attr_set = true;
    }
    PdlLaunch L(dim3((unsigned)pl.grid), dim3(TC_THREADS), pl.smem, st);
    CSD_CUDA(cudaLaunchKernelEx(&L.cfg, kern, tw, tw2, tx, rp));
    count_launch();
    return CSD_OK;
}

csd_status launch_linear_rs(const LinearArgs& a, cudaStream_t st) {
    const bool dual = a.W2 != nullptr;
    if (!rs_supported(a.m, a.N, a.K, dual)) return CSD_ERR_UNSUPPORTED;
    if (!a.xs || (((uintptr_t)a.xs) & 15)) return CSD_ERR_INVALID_ARG;
    const RsPlan pl = rs_plan(a.m, a.N, a.K, dual);
    CUtensorMap tw, tw2, tx;
    if (!tensor_map_2d(a.W, a.N, a.K, pl.box, &tw)) return CSD_ERR_UNSUPPORTED;
    tw2 = tw;
    if (dual && !tensor_map_2d(a.W2, a.N, a.K, pl.box, &tw2)) return CSD_ERR_UNSUPPORTED;
    if (!tensor_map_2d(a.xs, 3 * a.m, a.K, pl.npad, &tx)) return CSD_ERR_UNSUPPORTED;
    int ssq_cnt = a.ssq_cnt;
    if (!a.xs_ready) {
        const csd_status s = launch_split_rows(a, st);
        if (s != CSD_OK) return s;
        ssq_cnt = split_ssq_entries(a.K);
    }
    RsParams rp;
    rp.Y = a.Y; rp.status = status_word_device();
    rp.ssq_in = a.gain ? a.ssq : nullptr; rp.ssq_cnt = ssq_cnt;
    rp.out_xs = a.out_xs; rp.out_gain = a.out_gain; rp.out_ssq = a.out_ssq; rp.out_ld = a.out_ld;
    rp.N = a.N; rp.K = a.K; rp.ldy = a.ldy; rp.nks = pl.nks; rp.ks = pl.ks; rp.T = pl.T; rp.V = pl.V;
    rp.box = pl.box; rp.rows8 = pl.rows8; rp.stages = pl.stages; rp.qp = pl.qp; rp.chunks = pl.chunks; rp.tmem_cols = pl.tmem_cols; rp.epilogue = a.epilogue; rp.eps = a.eps;
#define CSD_RS_CASE(MM) \
    case MM: return dual ? launch_rs<MM, true>(tw, tw2, tx, rp, pl, st) : launch_rs<MM, false>(tw, tw2, tx, rp, pl, st);
    switch (a.m) {
        CSD_RS_CASE(1) CSD_RS_CASE(2) CSD_RS_CASE(3) CSD_RS_CASE(4) CSD_RS_CASE(5) CSD_RS_CASE(6) CSD_RS_CASE(7)
        CSD_RS_CASE(8) CSD_RS_CASE(9) CSD_RS_CASE(10) CSD_RS_CASE(11) CSD_RS_CASE(12) CSD_RS_CASE(13)
        CSD_RS_CASE(14) CSD_RS_CASE(15) CSD_RS_CASE(16) CSD_RS_CASE(17)
    }
#undef CSD_RS_CASE
    return CSD_ERR_INVALID_ARG;
}

}  // namespace csd
