// Tensor-core variant of the weight-streaming skinny GEMM  Y[m, N] = X[m, K] . W[N, K]^T.
//
// The weights are the wide operand: tiles of 128 weight rows x 64 K-elements arrive by TMA
// (128-byte swizzle) in a ring of shared-memory stages and are multiplied with tcgen05.mma
// (M = 128, K = 16 per instruction, fp32 accumulators in tensor memory).  The block's rows are
// the narrow operand.  To keep fp32 activations exact, every x is split into three bf16 terms
// x = b1 + b2 + b3 (8 + 8 + 8 mantissa bits); the three terms of the m rows are 3m columns of the
// narrow operand (padded to 16/32/48/64).  The split lives in global memory ([3m][K] bf16, written
// by the epilogue of the kernel that produced the rows, or by split_rows_kernel) and its 64-wide
// K block rides in the same stage as the weight tile; the epilogue adds the three partial results.
//
// Work is cut into (tile, K block) units and every CTA (one per SM) owns an equal contiguous share
// of them, so all SMs stream the same number of bytes; a tile that straddles CTAs is finished by
// the first of them (for which it comes last), adding the parts the others parked in CTA order
// (deterministic).  Roles inside a CTA (192 threads): warp 0 lane 0 issues TMA, warp 1 lane 0
// issues MMA, warps 2-5 read the accumulators from tensor memory (one quadrant each) and run the
// epilogue: rms-norm factor, residual add or gated activation, and optionally the three-term
// split and sum-of-squares pieces of the result for the next GEMM.  The first ring-full of weight
// tiles is requested before the programmatic-dependent-launch wait.  Every mbarrier wait is
// bounded; on a time-out the CTA records CSD_ERR_TIMEOUT, stops, frees its tensor memory, returns.
#include "gemm_tc.cuh"
#include "tc_common.cuh"
#include <mutex>
#include <unordered_map>

namespace csd {

constexpr size_t TC_SMEM_MAX = 111 * 1024;              // two CTAs (of consecutive kernels) fit one SM

static int g_path = 0;
void set_gemm_path(int path) { g_path = path; }
int gemm_path() { return g_path; }

static int npad_for(int m) { int c = 3 * m; return c <= 16 ? 16 : (c <= 32 ? 32 : (c <= 48 ? 48 : 64)); }

struct TcPlan {
    int npad, tiles, kblocks, grid, stages, csplit;    // kblocks: stages of work per tile (one or two 64-wide K blocks each)
    size_t smem, scratch_floats;
};

int tc_sm_count() {
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
    }
    return n;
}

// One CTA per SM; the (tile, K block) units are dealt out in equal contiguous shares.
static TcPlan tc_plan(int m, int N, int K, bool dual) {
    TcPlan p{};
    p.npad = npad_for(m);
    p.tiles = (N + TILE_N - 1) / TILE_N;
    p.kblocks = (K + KB - 1) / KB;
    // single-matrix GEMM on a block of up to 5 rows: a stage holds two K blocks (32 KB of weights per barrier
    // round trip, like the gated pair; measured 3-5 % faster per forward).  Larger blocks keep one K block per
    // stage, or too few stages would fit.
    const int ks = (!dual && p.npad <= 16) ? 2 : 1;
    p.kblocks = (p.kblocks + ks - 1) / ks;
    const long long units = (long long)p.tiles * p.kblocks;
    long long grid = units / 4;                           // at least four units per CTA
    if (grid < 1) grid = 1;
    if (grid > tc_sm_count()) grid = tc_sm_count();
    p.grid = (int)grid;
    // A single-matrix GEMM with few tiles (N = 4096: 32) on a block of up to 5 rows is cut the other way:
    // every tile goes to a cluster of four CTAs that share its K range and add their parts up through
    // distributed shared memory, on chip, instead of parking them in global memory.  4 x 32 = 128 streaming
    // SMs still draw the full bandwidth.  (Measured: 0.8 % faster per 7B forward at 5 rows, no gain at 9,
    // 1 % slower at 17, hence the row limit.)
    p.csplit = 1;
    if (!dual && p.npad <= 16 && p.tiles * 4 <= tc_sm_count() && p.tiles * 4 >= 96 && p.kblocks >= 8) {
        p.csplit = 4;
        p.grid = p.tiles * 4;
    }
    const size_t stage = (size_t)STAGE_BYTES * (dual ? 2 : ks) + (size_t)p.npad * 128 * ks;
    p.stages = (int)((TC_SMEM_MAX - 1024) / stage);
    if (p.stages > 12) p.stages = 12;
    p.smem = (size_t)p.stages * stage + 1024;
    p.scratch_floats = (size_t)p.grid * 2 * (dual ? 2 : 1) * m * TILE_N;
    return p;
}

bool tc_supported(int m, int N, int K, bool dual) {
    (void)dual;
    if (!(m >= 1 && m <= CSD_MAX_ROWS && N >= 1 && K >= 64 && (K & 7) == 0)) return false;
    const long long units = (long long)((N + TILE_N - 1) / TILE_N) * ((K + KB - 1) / KB);
    return units * (tc_sm_count() + 1) < (1LL << 31);
}

size_t tc_scratch_bytes(int m, int N, int K, bool dual) {
    if (!tc_supported(m, N, K, dual)) return 0;
    return align_up((size_t)tc_sm_count() * 2 * (dual ? 2 : 1) * m * TILE_N * sizeof(float), 256);
}

int tc_ticket_count(int N) { return (N + TILE_N - 1) / TILE_N + 1; }

// ---- tensor maps for the weight matrices (cached per pointer and shape) -------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

struct MapKey {
    const void* p; int N, K, box;
    bool operator==(const MapKey& o) const { return p == o.p && N == o.N && K == o.K && box == o.box; }
};
struct MapHash {
    size_t operator()(const MapKey& k) const { return (size_t)k.p ^ ((size_t)k.N << 20) ^ ((size_t)k.K << 40); }
};
static std::mutex g_map_mu;
static std::unordered_map<MapKey, CUtensorMap, MapHash> g_maps;

// [rows][K] bf16 row-major, boxes of box_rows x 64 elements, 128-byte swizzle, zero fill outside
bool tensor_map_2d(const void* W, int N, int K, int box_rows, CUtensorMap* out) {
    std::lock_guard<std::mutex> lk(g_map_mu);
    auto it = g_maps.find(MapKey{W, N, K, box_rows});
    if (it != g_maps.end()) { *out = it->second; return true; }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    CUtensorMap tm;
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)N};
    cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    cuuint32_t box[2] = {(cuuint32_t)KB, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(W), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return false;
    if (g_maps.size() > 4096) g_maps.clear();
    g_maps.emplace(MapKey{W, N, K, box_rows}, tm);
    *out = tm;
    return true;
}

struct TcParams {
    float* Y; float* partial; unsigned* tickets; int* status;
    const float* ssq_in; int ssq_cnt;                      // rms-norm: sum of squares of the input rows, in pieces
    __nv_bfloat16* out_xs; const __nv_bfloat16* out_gain; float* out_ssq; int out_ld;
    int N, K, ldy, nkb, tiles, stages, epilogue, csplit;
    float eps;
};

struct __align__(8) TcCtrl {
    uint64_t full[12], empty[12], acc_full[2], acc_empty[2];
    uint64_t red_ready, red_done;      // cluster split: the leader's buffer is free / all parts have been written
    uint32_t tmem_base;
    int abort_flag;
    float scale[32];
};

__device__ __forceinline__ float tc_gelu(float x) {
    return 0.5f * x * (1.f + tanhf(0.7978845608028654f * (x + 0.044715f * x * x * x)));
}
__device__ __forceinline__ float tc_silu(float x) { return x / (1.f + expf(-x)); }

// Units of work are (tile of 128 output columns, 64-wide K block) pairs in tile-major order; CTA c
// owns the contiguous range [unit_begin(c), unit_begin(c+1)), so every SM streams the same
// number of weight bytes whatever N and K are.
// (units * ctas fits 32 bits: the planner refuses shapes where it would not)
__device__ __forceinline__ unsigned unit_begin(unsigned c, unsigned units, unsigned ctas) { return c * units / ctas; }
__device__ __forceinline__ int cta_of_unit(unsigned u, unsigned units, unsigned ctas) {
    unsigned c = ((u + 1) * ctas - 1) / units;
    while (c + 1 < ctas && unit_begin(c + 1, units, ctas) <= u) ++c;
    while (c > 0 && unit_begin(c, units, ctas) > u) --c;
    return (int)c;
}

// ---- distributed shared memory (cluster split) ---------------------------------------------------
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void remote_arrive(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void remote_store(uint32_t cluster_addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(cluster_addr), "f"(v) : "memory");
}
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity) {   // acquire at cluster scope, bounded
    const uint32_t a = smem_u32(bar);
    for (int i = 0; i < SPIN_LIMIT; ++i) {
        uint32_t ok;
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                     : "=r"(ok) : "r"(a), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}

__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

template <int M, bool DUAL>
__global__ void __launch_bounds__(TC_THREADS, 2)
skinny_gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmW2,
                      const __grid_constant__ CUtensorMap tmX, const TcParams p) {
    constexpr int NPAD = 3 * M <= 16 ? 16 : (3 * M <= 32 ? 32 : (3 * M <= 48 ? 48 : 64));
    constexpr int NT = DUAL ? 2 : 1;
    constexpr int ACC_ONE = NPAD * NT;                        // tensor-memory columns of one accumulator
    // The tensor core's fp32 accumulation loses a little with every add of a long chain, so the K blocks
    // of a segment go round-robin to NACC accumulators (as many as fit 256 columns twice over, at most
    // 4); the epilogue adds them.
    constexpr int NACC = 2 * ACC_ONE * 4 <= 256 ? 4 : (2 * ACC_ONE * 2 <= 256 ? 2 : 1);
    constexpr int ACC_COLS = ACC_ONE * NACC;                  // columns per accumulator set (one segment)
    constexpr int TMEM_COLS = 2 * ACC_COLS <= 32 ? 32 : (2 * ACC_COLS <= 64 ? 64 : (2 * ACC_COLS <= 128 ? 128 : 256));
    constexpr int XBYTES = NPAD * 128;                        // the rows' terms for one K block
    constexpr int KS = (!DUAL && NPAD <= 16) ? 2 : 1;         // K blocks per stage
    constexpr int WB = (DUAL ? 2 : KS) * STAGE_BYTES;         // weight bytes per stage
    constexpr int STAGE = WB + KS * XBYTES;
    constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NPAD >> 3) << 17) |
                               ((uint32_t)(TILE_N >> 4) << 24);   // f32 accumulate, bf16 x bf16, K-major both

    extern __shared__ unsigned char smem_raw[];
    unsigned char* ring = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    TcCtrl* ctl = (TcCtrl*)(ring + (size_t)p.stages * STAGE);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x, ctas = gridDim.x;
    const unsigned units = (unsigned)p.tiles * (unsigned)p.nkb;
    unsigned u0 = unit_begin(cta, units, ctas), u1 = unit_begin(cta + 1, units, ctas);
    const int crank = p.csplit > 1 ? cta % p.csplit : 0;     // cluster split: rank inside the tile's cluster
    if (p.csplit > 1) {
        const unsigned t = (unsigned)(cta / p.csplit) * (unsigned)p.nkb;
        u0 = t + (unsigned)crank * (unsigned)p.nkb / (unsigned)p.csplit;
        u1 = t + (unsigned)(crank + 1) * (unsigned)p.nkb / (unsigned)p.csplit;
    }
    const int items = (int)(u1 - u0);

    if (tid == 0) {
        for (int s = 0; s < 12; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&ctl->acc_full[b], 1); mbar_init(&ctl->acc_empty[b], 4); }
        mbar_init(&ctl->red_ready, 1);
        mbar_init(&ctl->red_done, 4 * 3);               // one arrival per epilogue warp of the three other CTAs
        ctl->abort_flag = 0;
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
    if (p.csplit > 1) {      // nobody signals a barrier of another CTA before that CTA has initialised it
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    }
    // Let the next kernel in the stream start now: its CTAs take the second slot of each SM, set
    // themselves up and request their first weight tiles while this kernel is still streaming;
    // they touch nothing this kernel writes before their own dependency wait.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == 0) {
        // ---- TMA producer.  The weights do not depend on the kernel that produces the rows, so
        //      the first ring-full of weight tiles goes out before the dependency wait; the rows'
        //      terms follow after it.
        if (lane == 0) {
            // (all index arithmetic of this thread is incremental: a division per stage costs more
            // than the copy instructions it feeds)
            const int pre = items < p.stages ? items : p.stages;
            int tile = (int)(u0 / p.nkb), kb = (int)(u0 % p.nkb);
            const int kb0 = kb;
            for (int i = 0; i < pre; ++i) {
                unsigned char* dst = ring + (size_t)i * STAGE;
                mbar_expect_tx(&ctl->full[i], (uint32_t)STAGE);
                tma_load_2d(dst, &tmW, &ctl->full[i], kb * KS * KB, tile * TILE_N);
                if (DUAL) tma_load_2d(dst + STAGE_BYTES, &tmW2, &ctl->full[i], kb * KB, tile * TILE_N);
                if (KS == 2) tma_load_2d(dst + STAGE_BYTES, &tmW, &ctl->full[i], (kb * KS + 1) * KB, tile * TILE_N);   // past K: zero fill
                if (++kb == p.nkb) { kb = 0; ++tile; }
            }
            asm volatile("griddepcontrol.wait;" ::: "memory");
            int kx = kb0;
            for (int i = 0; i < pre; ++i) {
#pragma unroll
                for (int j = 0; j < KS; ++j)
                    tma_load_2d(ring + (size_t)i * STAGE + WB + j * XBYTES, &tmX, &ctl->full[i], (kx * KS + j) * KB, 0);
                if (++kx == p.nkb) kx = 0;
            }
            int s = 0;
            uint32_t ph = 0;                      // parity of the phase of empty[s] that frees slot s next
            for (int i = pre; i < items && !*abort_flag; ++i) {
                if (!mbar_wait(&ctl->empty[s], ph)) { *abort_flag = 1; break; }
                unsigned char* dst = ring + (size_t)s * STAGE;
                mbar_expect_tx(&ctl->full[s], (uint32_t)STAGE);
                tma_load_2d(dst, &tmW, &ctl->full[s], kb * KS * KB, tile * TILE_N);
                if (DUAL) tma_load_2d(dst + STAGE_BYTES, &tmW2, &ctl->full[s], kb * KB, tile * TILE_N);
                if (KS == 2) tma_load_2d(dst + STAGE_BYTES, &tmW, &ctl->full[s], (kb * KS + 1) * KB, tile * TILE_N);
#pragma unroll
                for (int j = 0; j < KS; ++j)
                    tma_load_2d(dst + WB + j * XBYTES, &tmX, &ctl->full[s], (kb * KS + j) * KB, 0);
                if (++kb == p.nkb) { kb = 0; ++tile; }
                if (++s == p.stages) { s = 0; ph ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer: one accumulator set per segment (the part of a tile inside this CTA's range)
        if (lane == 0) {
            int i = 0, s = 0;
            uint32_t ph = 0;                      // parity of the phase of full[s] that fills slot s next
            int kb_begin = (int)(u0 % p.nkb);
            const uint64_t desc0 = smem_desc_sw128(smem_u32(ring));   // descriptors differ in the address field only
            for (int seg = 0; i < items && !*abort_flag; ++seg) {
                const int b = seg & 1;
                const int seg_len = min(p.nkb - kb_begin, items - i);
                kb_begin = 0;                     // later segments start at a tile's first K block
                if (!mbar_wait(&ctl->acc_empty[b], ((seg >> 1) & 1) ^ 1)) { *abort_flag = 1; break; }
                tc_fence_after();
                const uint32_t dset = tmem + (uint32_t)(b * ACC_COLS);
                for (int j = 0; j < seg_len; ++j, ++i) {
                    const uint32_t d0 = dset + (uint32_t)((j % NACC) * ACC_ONE);
                    const int first = j < NACC ? 0 : 1;       // an accumulator's first K block overwrites it
                    if (!mbar_wait(&ctl->full[s], ph)) { *abort_flag = 1; break; }
                    tc_fence_after();
                    const uint64_t ad = desc0 + (uint64_t)(((uint32_t)s * (uint32_t)STAGE) >> 4);
                    const uint64_t bd = ad + (WB >> 4);
#pragma unroll
                    for (int h = 0; h < KS; ++h)
#pragma unroll
                        for (int k = 0; k < KB / 16; ++k) {
                            const uint64_t bdk = bd + ((h * XBYTES) >> 4) + 2 * k;
                            tc_mma(d0, ad + ((h * STAGE_BYTES) >> 4) + 2 * k, bdk, IDESC, (first | h | k) != 0);
                            if (DUAL) tc_mma(d0 + NPAD, ad + (STAGE_BYTES >> 4) + 2 * k, bdk, IDESC, (first | k) != 0);
                        }
                    tc_commit(&ctl->empty[s]);          // stage reusable once these MMAs have read it
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                }
                if (*abort_flag) break;
                tc_commit(&ctl->acc_full[b]);           // this segment's accumulators are complete
            }
        }
    } else {
        // ---- epilogue warps: quadrant q of tensor memory holds weight rows q*32 .. q*32+31 of the tile
        const int q = warp & 3, et = (warp - 2) * 32 + lane;
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (p.ssq_in && et < M) {               // rms-norm factor of every row from the pieces of its sum of squares
            float sq = 0.f;
            for (int c = 0; c < p.ssq_cnt; ++c) sq += __ldcg(p.ssq_in + (size_t)c * M + et);
            ctl->scale[et] = 1.f / sqrtf(sq / (float)p.K + p.eps);
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        float* my_part = p.partial + (size_t)cta * 2 * NT * M * TILE_N;
        int i = 0;
        for (int seg = 0; i < items; ++seg) {
            const int b = seg & 1;
            const int tile = (int)((u0 + i) / p.nkb), kb_begin = (int)((u0 + i) % p.nkb);
            const int seg_len = min(p.nkb - kb_begin, items - i);
            i += seg_len;
            if (!mbar_wait(&ctl->acc_full[b], (seg >> 1) & 1)) { *abort_flag = 1; break; }   // same outcome in all four warps
            tc_fence_after();
            const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * ACC_COLS);
            float sums[NT][M];
#pragma unroll
            for (int u = 0; u < NT; ++u) {
                float third[M], second[M];
#pragma unroll
                for (int r = 0; r < M; ++r) { sums[u][r] = 0.f; second[r] = 0.f; third[r] = 0.f; }
#pragma unroll
                for (int a = 0; a < NACC; ++a) {
                    if (a >= seg_len) break;            // a short segment used fewer accumulators
#pragma unroll
                    for (int c0 = 0; c0 < NPAD; c0 += 16) {
                        if (c0 >= 3 * M) break;
                        float v[16];
                        tc_ld16(taddr + (uint32_t)(a * ACC_ONE + u * NPAD + c0), v);
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            const int col = c0 + c;
                            if (col < M) sums[u][col] += v[c];
                            else if (col < 2 * M) second[col - M] += v[c];
                            else if (col < 3 * M) third[col - 2 * M] += v[c];
                        }
                    }
                }
#pragma unroll
                for (int r = 0; r < M; ++r) sums[u][r] += second[r] + third[r];   // small terms first
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->acc_empty[b]);
            const int col = q * 32 + lane, n = tile * TILE_N + col;
            // what the finishing step needs besides the sums is requested now, so that it travels while
            // the partial sums are parked and the ticket is taken (only the finisher uses it)
            float yold[M];
            float out_g = 1.f;
#pragma unroll
            for (int r = 0; r < M; ++r) yold[r] = 0.f;
            if (n < p.N) {
                if (p.epilogue == EPI_ADD) {
#pragma unroll
                    for (int r = 0; r < M; ++r) yold[r] = __ldcg(p.Y + (size_t)r * p.ldy + n);
                }
                if (p.out_xs && p.out_gain) out_g = __bfloat162float(p.out_gain[n]);
            }
            if (p.csplit > 1) {
                // Cluster split: the four CTAs of the cluster hold the four K ranges of this tile.  Rank 0
                // finishes the tile; when its own MMAs are done its ring is free, it tells the others, they
                // write their parts into it (distributed shared memory) and signal back, and it adds the
                // parts in rank order.
                constexpr int NV = NT * M;
                float* buf = reinterpret_cast<float*>(ring);          // [3][NV][128]
                if (crank == 0) {
                    if (et == 0)
                        for (int r = 1; r < p.csplit; ++r) remote_arrive(map_to_cta(smem_u32(&ctl->red_ready), (uint32_t)r));
                    if (!mbar_wait_cluster(&ctl->red_done, 0)) *abort_flag = 1;
#pragma unroll
                    for (int r = 1; r < 4; ++r)
#pragma unroll
                        for (int u = 0; u < NT; ++u)
#pragma unroll
                            for (int rr = 0; rr < M; ++rr) sums[u][rr] += buf[((r - 1) * NV + u * M + rr) * TILE_N + col];
                } else {
                    if (!mbar_wait_cluster(&ctl->red_ready, 0)) *abort_flag = 1;
                    const uint32_t dst = map_to_cta(smem_u32(buf), 0u);
#pragma unroll
                    for (int u = 0; u < NT; ++u)
#pragma unroll
                        for (int rr = 0; rr < M; ++rr)
                            remote_store(dst + (uint32_t)((((crank - 1) * NV + u * M + rr) * TILE_N + col) * 4), sums[u][rr]);
                    __syncwarp();
                    if (lane == 0) remote_arrive(map_to_cta(smem_u32(&ctl->red_done), 0u));
                    continue;
                }
            } else if (seg_len < p.nkb) {
                // Part of a tile.  Its contributors are consecutive CTAs; the first of them finishes it.
                // For the last contributor the tile is the FIRST thing it computes, so its partial sums
                // are parked in global memory (and its arrival counted) long before the first contributor,
                // for which the tile comes LAST, asks for them; a contributor whose whole share lies inside
                // the tile parks at the end, and the finisher waits for it (bounded).  Parts are added in
                // CTA order (deterministic).  Measured against "whoever arrives last finishes": 1.7 % faster
                // per forward at 5 rows, 4 % at 17; taking the first contributor's part of the tile first,
                // so that a middle contributor can finish without waiting, was slower again.
                const int c_lo = cta_of_unit((unsigned)tile * p.nkb, units, ctas);
                const int c_hi = cta_of_unit((unsigned)(tile + 1) * p.nkb - 1, units, ctas);
                if (cta != c_lo) {
                    float* mine = my_part;              // (a later contributor's part opens its share: slot 0)
#pragma unroll
                    for (int u = 0; u < NT; ++u)
#pragma unroll
                        for (int r = 0; r < M; ++r) mine[(u * M + r) * TILE_N + col] = sums[u][r];
                    __threadfence();
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (et == 0) atomicAdd(&p.tickets[tile], 1u);
                    continue;
                }
                if (et == 0) {
                    const unsigned want = (unsigned)(c_hi - c_lo);
                    int spins = 0;
                    while (ld_acquire_gpu(&p.tickets[tile]) < want) {
                        if (++spins > SPIN_LIMIT) { *abort_flag = 1; break; }
                    }
                    p.tickets[tile] = 0u;               // everyone has arrived: ready for the next launch
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
                __threadfence();
                // the other parts in CTA order; as many contributors' loads in flight together as about 48
                // registers hold (all of them, in one round trip, for a 5-row block)
                constexpr int NV = NT * M, CH = NV <= 6 ? 8 : (48 / NV < 1 ? 1 : 48 / NV);
                for (int c = c_lo + 1; c <= c_hi; c += CH) {
                    float part[CH][NV];
#pragma unroll
                    for (int h = 0; h < CH; ++h) {
                        const int cc = min(c + h, c_hi);
                        const float* src = p.partial + ((size_t)cc * 2) * NT * M * TILE_N + col;
#pragma unroll
                        for (int v = 0; v < NV; ++v) part[h][v] = __ldcg(src + v * TILE_N);
                    }
#pragma unroll
                    for (int h = 0; h < CH; ++h)
                        if (c + h <= c_hi) {
#pragma unroll
                            for (int u = 0; u < NT; ++u)
#pragma unroll
                                for (int r = 0; r < M; ++r) sums[u][r] += part[h][u * M + r];
                        }
                }
            }
            // ---- finish the tile: this thread owns output column n for all M rows
            float outv[M];
#pragma unroll
            for (int r = 0; r < M; ++r) {
                const float scale = p.ssq_in ? ctl->scale[r] : 1.f;
                float val = sums[0][r] * scale;
                if (DUAL) {
                    const float up = sums[NT - 1][r] * scale;
                    val = (p.epilogue == EPI_GEGLU ? tc_gelu(val) : tc_silu(val)) * up;
                }
                if (n < p.N) {
                    float* y = p.Y + (size_t)r * p.ldy + n;
                    if (p.epilogue == EPI_ADD) val += yold[r];
                    *y = val;
                } else {
                    val = 0.f;
                }
                outv[r] = val;
            }
            if (p.out_ssq) {                      // pieces of the rows' sums of squares, one per 32 columns
#pragma unroll
                for (int r = 0; r < M; ++r) {
                    const float sq = warp_sum(outv[r] * outv[r]);
                    if (lane == 0) p.out_ssq[(size_t)(tile * 4 + q) * M + r] = sq;
                }
            }
            if (p.out_xs && n < p.N) {            // the rows as three bf16 terms for the GEMM that reads them next
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
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

// Stand-alone split of fp32 rows (times an optional gain) into three bf16 terms, plus the pieces of
// each row's sum of squares.  grid = (K / 1024 rounded up, m).
__global__ void __launch_bounds__(128)
split_rows_kernel(const float* __restrict__ X, int ldx, int K, int m, const __nv_bfloat16* __restrict__ gain,
                  __nv_bfloat16* __restrict__ xs, float* __restrict__ ssq) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int r = blockIdx.y, k = (blockIdx.x * 128 + threadIdx.x) * 8;
    float sq = 0.f;
    if (k < K) {
        const float* src = X + (size_t)r * ldx + k;
        const float4 a = *reinterpret_cast<const float4*>(src), b = *reinterpret_cast<const float4*>(src + 4);
        float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
        for (int e = 0; e < 8; ++e) sq = fmaf(v[e], v[e], sq);
        if (gain) {
            const uint4 g = *reinterpret_cast<const uint4*>(gain + k);
            v[0] *= bf16lo(g.x); v[1] *= bf16hi(g.x); v[2] *= bf16lo(g.y); v[3] *= bf16hi(g.y);
            v[4] *= bf16lo(g.z); v[5] *= bf16hi(g.z); v[6] *= bf16lo(g.w); v[7] *= bf16hi(g.w);
        }
        uint32_t t[3][4];
#pragma unroll
        for (int e = 0; e < 8; e += 2) {
            uint16_t a1, a2, a3, c1, c2, c3;
            split3(v[e], a1, a2, a3);
            split3(v[e + 1], c1, c2, c3);
            t[0][e / 2] = a1 | ((uint32_t)c1 << 16); t[1][e / 2] = a2 | ((uint32_t)c2 << 16);
            t[2][e / 2] = a3 | ((uint32_t)c3 << 16);
        }
#pragma unroll
        for (int s = 0; s < 3; ++s)
            *reinterpret_cast<uint4*>(xs + (size_t)(s * m + r) * K + k) = make_uint4(t[s][0], t[s][1], t[s][2], t[s][3]);
    }
    __shared__ float part[4];
    sq = warp_sum(sq);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = sq;
    __syncthreads();
    if (threadIdx.x == 0 && ssq) ssq[(size_t)blockIdx.x * m + r] = (part[0] + part[1]) + (part[2] + part[3]);
}

int split_rows(int m) { return npad_for(m); }
int split_ssq_entries(int K) { return (K + 1023) / 1024; }

static void pdl_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute* attr, dim3 grid, dim3 block, size_t smem,
                       cudaStream_t st) {
    cfg = cudaLaunchConfig_t{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
}

// Splits a.X (times a.gain) into a.xs and writes the sum-of-squares pieces into a.ssq.
csd_status launch_split_rows(const LinearArgs& a, cudaStream_t st) {
    if (!a.X || (((uintptr_t)a.X) & 15) || (a.ldx & 3)) return CSD_ERR_INVALID_ARG;
    if (a.gain && !a.ssq) return CSD_ERR_INVALID_ARG;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    pdl_config(cfg, attr, dim3((unsigned)split_ssq_entries(a.K), (unsigned)a.m), dim3(128), 0, st);
    CSD_CUDA(cudaLaunchKernelEx(&cfg, split_rows_kernel, a.X, a.ldx, a.K, a.m, a.gain, a.xs,
                                a.gain ? a.ssq : (float*)nullptr));
    count_launch();
    return CSD_OK;
}

template <int M, bool DUAL>
static csd_status launch_tc(const CUtensorMap& tw, const CUtensorMap& tw2, const CUtensorMap& tx, const TcParams& tp,
                            const TcPlan& pl, cudaStream_t st) {
    auto kern = skinny_gemm_tc_kernel<M, DUAL>;
    static bool attr_set = false;
    if (!attr_set) {
        CSD_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM_MAX + 1024));
        // ask for the largest shared-memory carve-out, or the second CTA (the next kernel's) does not fit
        CSD_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
        attr_set = true;
    }
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    pdl_config(cfg, attr, dim3((unsigned)pl.grid), dim3(TC_THREADS), pl.smem + 1024, st);
    if (pl.csplit > 1) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)pl.csplit; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    CSD_CUDA(cudaLaunchKernelEx(&cfg, kern, tw, tw2, tx, tp));
    count_launch();
    return CSD_OK;
}

csd_status launch_linear_tc(const LinearArgs& a, cudaStream_t st) {
    const bool dual = a.W2 != nullptr;
    if (!tc_supported(a.m, a.N, a.K, dual)) return CSD_ERR_UNSUPPORTED;
    if (!a.xs || !a.partial || !a.tickets) return CSD_ERR_INVALID_ARG;
    if ((((uintptr_t)a.xs) & 15)) return CSD_ERR_INVALID_ARG;
    const TcPlan pl = tc_plan(a.m, a.N, a.K, dual);
    CUtensorMap tw, tw2, tx;
    if (!tensor_map_2d(a.W, a.N, a.K, TILE_N, &tw)) return CSD_ERR_UNSUPPORTED;
    tw2 = tw;
    if (dual && !tensor_map_2d(a.W2, a.N, a.K, TILE_N, &tw2)) return CSD_ERR_UNSUPPORTED;
    if (!tensor_map_2d(a.xs, 3 * a.m, a.K, pl.npad, &tx)) return CSD_ERR_UNSUPPORTED;
    int ssq_cnt = a.ssq_cnt;
    if (!a.xs_ready) {
        const csd_status s = launch_split_rows(a, st);
        if (s != CSD_OK) return s;
        ssq_cnt = split_ssq_entries(a.K);
    }
    TcParams tp;
    tp.Y = a.Y; tp.partial = a.partial; tp.tickets = a.tickets; tp.status = status_word_device();
    tp.ssq_in = a.gain ? a.ssq : nullptr; tp.ssq_cnt = ssq_cnt;
    tp.out_xs = a.out_xs; tp.out_gain = a.out_gain; tp.out_ssq = a.out_ssq; tp.out_ld = a.out_ld;
    tp.N = a.N; tp.K = a.K; tp.ldy = a.ldy; tp.nkb = pl.kblocks; tp.tiles = pl.tiles; tp.stages = pl.stages; tp.csplit = pl.csplit;
    tp.epilogue = a.epilogue; tp.eps = a.eps;
#define CSD_TC_CASE(MM) \
    case MM: return dual ? launch_tc<MM, true>(tw, tw2, tx, tp, pl, st) : launch_tc<MM, false>(tw, tw2, tx, tp, pl, st);
    switch (a.m) {
        CSD_TC_CASE(1) CSD_TC_CASE(2) CSD_TC_CASE(3) CSD_TC_CASE(4) CSD_TC_CASE(5) CSD_TC_CASE(6) CSD_TC_CASE(7)
        CSD_TC_CASE(8) CSD_TC_CASE(9) CSD_TC_CASE(10) CSD_TC_CASE(11) CSD_TC_CASE(12) CSD_TC_CASE(13)
        CSD_TC_CASE(14) CSD_TC_CASE(15) CSD_TC_CASE(16) CSD_TC_CASE(17)
    }
#undef CSD_TC_CASE
    return CSD_ERR_INVALID_ARG;
}

}  // namespace csd
