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
#include <string.h>

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
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {   // one poll; test_wait never suspends the thread, so the other cursor keeps moving
    uint32_t ok;
    asm volatile("{ .reg .pred p; mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
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

template <int M>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_chain_kernel(const __grid_constant__ ChainParams cp) {
    constexpr int NPAD = 3 * M <= 16 ? 16 : (3 * M <= 32 ? 32 : (3 * M <= 48 ? 48 : 64));
    constexpr int ACC_COLS = 2 * NPAD;                         // room for the two matrices of a gated GEMM
    constexpr int TMEM_COLS = 2 * ACC_COLS <= 64 ? 64 : (2 * ACC_COLS <= 128 ? 128 : 256);
    constexpr int XBYTES = NPAD * 128;
    constexpr int STAGE = STAGE_BYTES + XBYTES;
    constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NPAD >> 3) << 17) |
                               ((uint32_t)(TILE_N >> 4) << 24);

    extern __shared__ unsigned char smem_raw[];
    unsigned char* ring = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    ChainCtrl* ctl = (ChainCtrl*)(ring + (size_t)cp.stages * STAGE);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const unsigned cta = blockIdx.x, ctas = gridDim.x;

    if (tid == 0) {
        for (int s = 0; s < 12; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&ctl->acc_full[b], 1); mbar_init(&ctl->acc_empty[b], 4); }
        ctl->abort_flag = 0; ctl->last_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&ctl->tmem_base)), "r"((uint32_t)TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctl->tmem_base;
    volatile int* abort_flag = &ctl->abort_flag;

    // this CTA's share of every GEMM of the chain
    // (a GEMM with fewer units than CTAs is shared among its first `eff` CTAs only, so that every
    // CTA between two that share a tile holds a part of it: the fix-up counts on that)
    unsigned u0[CHAIN_MAX_OPS], cnt[CHAIN_MAX_OPS], units[CHAIN_MAX_OPS], eff[CHAIN_MAX_OPS];
    int total = 0;
#pragma unroll
    for (int j = 0; j < CHAIN_MAX_OPS; ++j) {
        u0[j] = cnt[j] = units[j] = 0;
        eff[j] = 1;
        if (j < cp.n_ops) {
            units[j] = (unsigned)cp.op[j].tiles * (unsigned)cp.op[j].nkb * (cp.op[j].dual ? 2u : 1u);
            eff[j] = units[j] < ctas ? units[j] : ctas;
            if (cta < eff[j]) {
                u0[j] = ch_unit_begin(cta, units[j], eff[j]);
                cnt[j] = ch_unit_begin(cta + 1, units[j], eff[j]) - u0[j];
            }
            total += (int)cnt[j];
        }
    }

    if (warp == 0) {
        // ---- TMA producer: two cursors over this CTA's items of all GEMMs.  Weight tiles run
        //      ahead as far as the ring allows; the rows' terms of GEMM j follow once GEMM j-1
        //      has been reported finished by every CTA.
        if (lane == 0) {
            int gw = 0, wop = 0; unsigned wi = 0;      // next weight tile: global index, GEMM, index inside it
            int gx = 0, xop = 0; unsigned xi = 0;      // next rows tile
            int dep_ok_upto = 0;                       // rows of GEMMs <= this index may be loaded
            int idle = 0;
            while (wop < cp.n_ops && cnt[wop] == 0) ++wop;
            while (xop < cp.n_ops && cnt[xop] == 0) ++xop;
            while (gx < total && !*abort_flag) {
                bool progressed = false;
                if (gw < total) {
                    const int s = gw % cp.stages;
                    if (gw < cp.stages || mbar_test(&ctl->empty[s], ((gw / cp.stages) - 1) & 1)) {
                        const ChainOpDev& o = cp.op[wop];
                        const UnitPos up = unit_pos(o, u0[wop] + wi);
                        mbar_expect_tx(&ctl->full[s], (uint32_t)STAGE);
                        tma_load_2d(ring + (size_t)s * STAGE, up.which ? &o.tmW2 : &o.tmW, &ctl->full[s], up.kb * KB,
                                    up.tile * TILE_N);
                        ++gw;
                        if (++wi == cnt[wop]) { wi = 0; do { ++wop; } while (wop < cp.n_ops && cnt[wop] == 0); }
                        progressed = true;
                    }
                }
                if (gx < gw) {
                    if (xop > dep_ok_upto) {
                        // GEMM xop reads what GEMM xop-1 wrote: has every CTA finished xop-1 ?
                        if ((int)(ld_acquire(cp.done + (xop - 1)) - cp.done_target) >= 0) {
                            // the rows were written with ordinary stores; the loads below go through the async proxy
                            asm volatile("fence.proxy.async.global;" ::: "memory");
                            dep_ok_upto = xop;
                        }
                    }
                    if (xop <= dep_ok_upto) {
                        const ChainOpDev& o = cp.op[xop];
                        const UnitPos up = unit_pos(o, u0[xop] + xi);
                        const int s = gx % cp.stages;
                        tma_load_2d(ring + (size_t)s * STAGE + STAGE_BYTES, &o.tmX, &ctl->full[s], up.kb * KB, 0);
                        ++gx;
                        if (++xi == cnt[xop]) { xi = 0; do { ++xop; } while (xop < cp.n_ops && cnt[xop] == 0); }
                        progressed = true;
                    }
                }
                if (progressed) idle = 0;
                else if (++idle > DEP_POLL_LIMIT) { *abort_flag = 1; break; }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer: one accumulator set per segment (the part of a tile inside this CTA's share)
        if (lane == 0) {
            int gi = 0, seg = 0;
            for (int j = 0; j < cp.n_ops && !*abort_flag; ++j) {
                const ChainOpDev& o = cp.op[j];
                const int per_tile = o.nkb * (o.dual ? 2 : 1);
                unsigned i = 0;
                while (i < cnt[j] && !*abort_flag) {
                    const int b = seg & 1;
                    const int rem = (int)((u0[j] + i) % per_tile);
                    const int seg_len = min(per_tile - rem, (int)(cnt[j] - i));
                    if (!mbar_wait(&ctl->acc_empty[b], ((seg >> 1) & 1) ^ 1)) { *abort_flag = 1; break; }
                    tc_fence_after();
                    const uint32_t d0 = tmem + (uint32_t)(b * ACC_COLS);
                    bool started[2] = {false, false};
                    for (int t = 0; t < seg_len; ++t, ++i, ++gi) {
                        const int s = gi % cp.stages;
                        if (!mbar_wait(&ctl->full[s], (gi / cp.stages) & 1)) { *abort_flag = 1; break; }
                        tc_fence_after();
                        const int which = o.dual ? (rem + t) & 1 : 0;
                        const uint32_t a_addr = smem_u32(ring + (size_t)s * STAGE);
                        const uint32_t b_addr = a_addr + STAGE_BYTES;
#pragma unroll
                        for (int k = 0; k < KB / 16; ++k)
                            tc_mma(d0 + which * NPAD, smem_desc_sw128(a_addr + k * 32), smem_desc_sw128(b_addr + k * 32),
                                   IDESC, (started[which] || k != 0) ? 1u : 0u);
                        started[which] = true;
                        tc_commit(&ctl->empty[s]);
                    }
                    if (*abort_flag) break;
                    tc_commit(&ctl->acc_full[b]);
                    ++seg;
                }
            }
        }
    } else {
        // ---- epilogue warps: quadrant q of tensor memory holds weight rows q*32 .. q*32+31 of the tile
        const int q = warp & 3, et = (warp - 2) * 32 + lane;
        float* my_part = cp.partial + (size_t)cta * 2 * 2 * M * TILE_N;
        int seg = 0;
        bool dead = false;
        for (int j = 0; j < cp.n_ops && !dead; ++j) {
            const ChainOpDev& o = cp.op[j];
            const int NT = o.dual ? 2 : 1, per_tile = o.nkb * NT;
            unsigned i = 0;
            int op_seg = 0;
            while (i < cnt[j]) {
                const int b = seg & 1;
                const int tile = (int)((u0[j] + i) / per_tile), rem = (int)((u0[j] + i) % per_tile);
                const int seg_len = min(per_tile - rem, (int)(cnt[j] - i));
                i += seg_len;
                if (!mbar_wait(&ctl->acc_full[b], (seg >> 1) & 1)) { *abort_flag = 1; dead = true; break; }
                tc_fence_after();
                if (op_seg == 0) {      // the rows of this GEMM are final by now: their rms-norm factors
                    if (o.ssq_in && et < M) {
                        float sq = 0.f;
                        for (int c = 0; c < o.ssq_cnt; ++c) sq += __ldcg(o.ssq_in + (size_t)c * M + et);
                        ctl->scale[et] = 1.f / sqrtf(sq / (float)o.K + o.eps);
                    }
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                }
                // which of the two matrices of a gated GEMM this segment touched at all
                const bool has0 = !o.dual || seg_len > 1 || (rem & 1) == 0;
                const bool has1 = o.dual && (seg_len > 1 || (rem & 1) == 1);
                const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * ACC_COLS);
                float sums[2][M];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
#pragma unroll
                    for (int r = 0; r < M; ++r) sums[u][r] = 0.f;
                    if (u == 0 ? !has0 : !has1) continue;
                    float third[M], second[M];
#pragma unroll
                    for (int r = 0; r < M; ++r) { second[r] = 0.f; third[r] = 0.f; }
#pragma unroll
                    for (int c0 = 0; c0 < NPAD; c0 += 16) {
                        if (c0 >= 3 * M) break;
                        float v[16];
                        tc_ld16(taddr + (uint32_t)(u * NPAD + c0), v);
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            const int col = c0 + c;
                            if (col < M) sums[u][col] = v[c];
                            else if (col < 2 * M) second[col - M] = v[c];
                            else if (col < 3 * M) third[col - 2 * M] = v[c];
                        }
                    }
#pragma unroll
                    for (int r = 0; r < M; ++r) sums[u][r] += second[r] + third[r];
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->acc_empty[b]);
                const int col = q * 32 + lane, n = tile * TILE_N + col;
                if (seg_len < per_tile) {
                    // part of a tile: park it (slot 0 = this CTA's first segment of the GEMM, 1 = a later
                    // one); whoever arrives last adds all parts in CTA order and finishes the tile
                    float* mine = my_part + (size_t)(op_seg == 0 ? 0 : 1) * 2 * M * TILE_N;
#pragma unroll
                    for (int u = 0; u < 2; ++u)
                        if (u < NT) {
#pragma unroll
                            for (int r = 0; r < M; ++r) mine[(u * M + r) * TILE_N + col] = sums[u][r];
                        }
                    __threadfence();
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    const int c_lo = ch_cta_of_unit((unsigned)tile * per_tile, units[j], eff[j]);
                    const int c_hi = ch_cta_of_unit((unsigned)(tile + 1) * per_tile - 1, units[j], eff[j]);
                    if (et == 0) {
                        const unsigned old = atomicAdd(&o.tickets[tile], 1u);
                        ctl->last_flag = (old == (unsigned)(c_hi - c_lo));
                        if (ctl->last_flag) o.tickets[tile] = 0u;
                    }
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    const int last = ctl->last_flag;
                    ++seg; ++op_seg;
                    if (!last) continue;
                    __threadfence();
#pragma unroll
                    for (int u = 0; u < 2; ++u)
#pragma unroll
                        for (int r = 0; r < M; ++r) sums[u][r] = 0.f;
                    for (int c = c_lo; c <= c_hi; ++c) {
                        const int slot = (int)(ch_unit_begin(c, units[j], eff[j]) / per_tile) == tile ? 0 : 1;
                        const float* src = cp.partial + ((size_t)c * 2 + slot) * 2 * M * TILE_N + col;
                        float part[2][M];
#pragma unroll
                        for (int u = 0; u < 2; ++u)
                            if (u < NT) {
#pragma unroll
                                for (int r = 0; r < M; ++r) part[u][r] = __ldcg(src + (u * M + r) * TILE_N);
                            }
#pragma unroll
                        for (int u = 0; u < 2; ++u)
                            if (u < NT) {
#pragma unroll
                                for (int r = 0; r < M; ++r) sums[u][r] += part[u][r];
                            }
                    }
                } else {
                    ++seg; ++op_seg;
                }
                // ---- finish the tile: this thread owns output column n for all M rows
                float outv[M];
#pragma unroll
                for (int r = 0; r < M; ++r) {
                    const float scale = o.ssq_in ? ctl->scale[r] : 1.f;
                    float val = sums[0][r] * scale;
                    if (o.dual) {
                        const float up = sums[1][r] * scale;
                        val = (o.epilogue == EPI_GEGLU ? ch_gelu(val) : ch_silu(val)) * up;
                    }
                    if (n < o.N) {
                        float* y = o.Y + (size_t)r * o.ldy + n;
                        if (o.epilogue == EPI_ADD) val += __ldcg(y);      // may have been written by another CTA of this launch
                        *y = val;
                    } else {
                        val = 0.f;
                    }
                    outv[r] = val;
                }
                if (o.out_ssq) {
#pragma unroll
                    for (int r = 0; r < M; ++r) {
                        const float sq = warp_sum(outv[r] * outv[r]);
                        if (lane == 0) o.out_ssq[(size_t)(tile * 4 + q) * M + r] = sq;
                    }
                }
                if (o.out_xs && n < o.N) {
                    const float g = o.out_gain ? __bfloat162float(o.out_gain[n]) : 1.f;
#pragma unroll
                    for (int r = 0; r < M; ++r) {
                        uint16_t b1, b2, b3;
                        split3(outv[r] * g, b1, b2, b3);
                        uint16_t* dst = reinterpret_cast<uint16_t*>(o.out_xs) + n;
                        dst[(size_t)r * o.out_ld] = b1;
                        dst[(size_t)(M + r) * o.out_ld] = b2;
                        dst[(size_t)(2 * M + r) * o.out_ld] = b3;
                    }
                }
            }
            if (dead) break;
            // report this GEMM finished by this CTA (its own tiles and any fix-ups it performed)
            __threadfence();
            asm volatile("fence.proxy.async.global;" ::: "memory");
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (et == 0) atomicAdd(cp.done + j, 1u);
        }
    }
    if (*abort_flag) {
        if (tid == 0) set_status(cp.status, CSD_ERR_TIMEOUT);
        __nanosleep(2000000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

static int chain_npad(int m) { int c = 3 * m; return c <= 16 ? 16 : (c <= 32 ? 32 : (c <= 48 ? 48 : 64)); }

size_t chain_scratch_bytes(int m) {
    return align_up((size_t)tc_sm_count() * 2 * 2 * m * TILE_N * sizeof(float), 256);
}

template <int M>
static csd_status launch_chain_m(const ChainParams& cp, int grid, size_t smem, cudaStream_t st) {
    auto kern = gemm_chain_kernel<M>;
    static bool attr_set = false;
    if (!attr_set) {
        CSD_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)CHAIN_SMEM + 1024));
        CSD_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
        attr_set = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(TC_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;      // every CTA resident at once: they wait for one another
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    CSD_CUDA(cudaLaunchKernelEx(&cfg, kern, cp));
    count_launch();
    return CSD_OK;
}

// ops[j+1] must read (a.xs) what ops[j] writes (a.out_xs); ops[0].xs must be ready.  done_dev:
// CHAIN_MAX_OPS zero-initialised counters owned by the caller, epoch_host: launches so far.
csd_status launch_linear_chain(const LinearArgs* ops, int n_ops, unsigned* done_dev, unsigned* epoch_host,
                               cudaStream_t st) {
    if (!ops || n_ops < 1 || n_ops > CHAIN_MAX_OPS || !done_dev || !epoch_host) return CSD_ERR_INVALID_ARG;
    const int m = ops[0].m, grid = tc_sm_count();
    if (m < 1 || m > CSD_MAX_ROWS) return CSD_ERR_INVALID_ARG;
    const int npad = chain_npad(m);
    ChainParams cp;
    memset(&cp, 0, sizeof(cp));
    size_t ticket_off = 0;
    for (int j = 0; j < n_ops; ++j) {
        const LinearArgs& a = ops[j];
        const bool dual = a.W2 != nullptr;
        if (a.m != m || !a.W || !a.Y || !a.xs || !a.partial || !a.tickets) return CSD_ERR_INVALID_ARG;
        if (j == 0 && !a.xs_ready) return CSD_ERR_INVALID_ARG;
        if (!tc_supported(a.m, a.N, a.K, dual)) return CSD_ERR_UNSUPPORTED;
        if (dual != (a.epilogue == EPI_SWIGLU || a.epilogue == EPI_GEGLU)) return CSD_ERR_INVALID_ARG;
        ChainOpDev& o = cp.op[j];
        o.tiles = (a.N + TILE_N - 1) / TILE_N;
        o.nkb = (a.K + KB - 1) / KB;
        if ((long long)o.tiles * o.nkb * (dual ? 2 : 1) * (grid + 1) >= (1LL << 31)) return CSD_ERR_UNSUPPORTED;
        if (!tensor_map_2d(a.W, a.N, a.K, TILE_N, &o.tmW)) return CSD_ERR_UNSUPPORTED;
        o.tmW2 = o.tmW;
        if (dual && !tensor_map_2d(a.W2, a.N, a.K, TILE_N, &o.tmW2)) return CSD_ERR_UNSUPPORTED;
        if (!tensor_map_2d(a.xs, 3 * m, a.K, npad, &o.tmX)) return CSD_ERR_UNSUPPORTED;
        o.Y = a.Y; o.ssq_in = a.gain ? a.ssq : nullptr; o.ssq_cnt = a.ssq_cnt;
        o.out_xs = a.out_xs; o.out_gain = a.out_gain; o.out_ssq = a.out_ssq; o.out_ld = a.out_ld;
        o.tickets = ops[0].tickets + ticket_off;
        ticket_off += (size_t)o.tiles;
        o.N = a.N; o.K = a.K; o.ldy = a.ldy; o.epilogue = a.epilogue; o.dual = dual ? 1 : 0; o.eps = a.eps;
    }
    cp.partial = ops[0].partial;
    cp.done = done_dev;
    cp.status = status_word_device();
    *epoch_host += 1;
    cp.done_target = *epoch_host * (unsigned)grid;
    cp.n_ops = n_ops;
    const size_t stage = (size_t)STAGE_BYTES + (size_t)npad * 128;
    int stages = (int)((CHAIN_SMEM - 2048) / stage);
    if (stages > 12) stages = 12;
    cp.stages = stages;
    const size_t smem = (size_t)stages * stage + 2048 + 1024;
#define CSD_CH_CASE(MM) case MM: return launch_chain_m<MM>(cp, grid, smem, st);
    switch (m) {
        CSD_CH_CASE(1) CSD_CH_CASE(2) CSD_CH_CASE(3) CSD_CH_CASE(4) CSD_CH_CASE(5) CSD_CH_CASE(6) CSD_CH_CASE(7)
        CSD_CH_CASE(8) CSD_CH_CASE(9) CSD_CH_CASE(10) CSD_CH_CASE(11) CSD_CH_CASE(12) CSD_CH_CASE(13)
        CSD_CH_CASE(14) CSD_CH_CASE(15) CSD_CH_CASE(16) CSD_CH_CASE(17)
    }
#undef CSD_CH_CASE
    return CSD_ERR_INVALID_ARG;
}

}  // namespace csd
