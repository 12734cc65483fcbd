// Tensor-core variant of the weight-streaming skinny GEMM  Y[m, N] = X[m, K] . W[N, K]^T.
//
// The weights are the wide operand: a CTA streams tiles of 128 weight rows x 64 K-elements with
// TMA (128-byte swizzle) through a ring of shared-memory stages and multiplies them with
// tcgen05.mma (M = 128, K = 16 per instruction, fp32 accumulators in tensor memory).  The block's
// rows are the narrow operand.  To keep fp32 activations exact, every x is split into three bf16
// terms x = b1 + b2 + b3 (8 + 8 + 8 mantissa bits); the three terms of the m rows are 3m columns
// of the narrow operand (padded to 16/32/48/64), kept resident in shared memory for the CTA's K
// slice, and the epilogue adds the three partial results.
//
// Roles inside a CTA (192 threads): warp 0 lane 0 issues TMA, warp 1 lane 0 issues MMA, warps 2-5
// read the accumulators from tensor memory (one quadrant each) and run the epilogue.  A CTA owns
// one K slice and walks over tiles of 128 output columns; with several K slices the partial sums
// go through scratch and the CTA that arrives last at the tile's ticket adds them in slice order
// and finishes the tile.  Every wait on an mbarrier is bounded; on a time-out the CTA records
// CSD_ERR_TIMEOUT, stops issuing work, releases its tensor memory and returns.
#include "gemm_tc.cuh"
#include <cuda.h>
#include <mutex>
#include <unordered_map>

namespace csd {

constexpr int TC_THREADS = 192;
constexpr int TILE_N = 128;       // weight rows per MMA (its M dimension)
constexpr int KB = 64;            // K elements per stage (one 128-byte swizzle atom wide)
constexpr int STAGE_BYTES = TILE_N * KB * 2;      // 16 KB
constexpr int SPIN_LIMIT = 20000000;              // bounded waits (about a second)
constexpr size_t TC_SMEM_MAX = 220 * 1024;

static int g_path = 0;
void set_gemm_path(int path) { g_path = path; }
int gemm_path() { return g_path; }

static int npad_for(int m) { int c = 3 * m; return c <= 16 ? 16 : (c <= 32 ? 32 : (c <= 48 ? 48 : 64)); }

struct TcPlan {
    int npad, tiles, kblocks, kb_per, kslices, grid, stages;
    size_t smem, x_bytes, scratch_floats;
};

static int tc_sm_count() {
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
    }
    return n;
}

// One K slice per CTA, resident split-X for that slice, as many ring stages as fit.  The slice
// count is chosen to minimise the predicted makespan: rounds of tiles per CTA times the slice
// length (plus a fixed cost per tile for the accumulator read-out).
static TcPlan tc_plan(int m, int N, int K, bool dual) {
    TcPlan best{};
    double best_cost = 1e300;
    const int npad = npad_for(m), sms = tc_sm_count();
    const int tiles = (N + TILE_N - 1) / TILE_N, kblocks = (K + KB - 1) / KB;
    const int stage = STAGE_BYTES * (dual ? 2 : 1);
    for (int ks = 1; ks <= 32 && ks <= kblocks; ++ks) {
        const int per = (kblocks + ks - 1) / ks;
        const int slices = (kblocks + per - 1) / per;
        if (slices != ks) continue;
        const size_t xb = (size_t)npad * per * KB * 2;
        if (xb + 2 * (size_t)stage + 2048 > TC_SMEM_MAX) continue;
        int stages = (int)((TC_SMEM_MAX - 2048 - xb) / stage);
        if (stages > 8) stages = 8;
        int ctas_per_slice = sms / ks;
        if (ctas_per_slice < 1) continue;
        if (ctas_per_slice > tiles) ctas_per_slice = tiles;
        const int rounds = (tiles + ctas_per_slice - 1) / ctas_per_slice;
        // time in units of one k-block streamed by one SM: the slice of every tile, an accumulator
        // read-out per tile, the split of this slice of X (exposed before the first MMA), and a
        // penalty when the ring is too shallow to cover the memory latency
        double cost = (double)rounds * (per + 1.5) + 0.06 * m * per + (ks > 1 ? 1.0 : 0.0);
        if (stages < 6) cost *= 1.0 + 0.25 * (6 - stages);
        if (cost < best_cost) {
            best_cost = cost;
            best.npad = npad; best.tiles = tiles; best.kblocks = kblocks; best.kb_per = per; best.kslices = ks;
            best.grid = ctas_per_slice * ks; best.stages = stages; best.x_bytes = xb;
            best.smem = xb + (size_t)stages * stage + 2048;
            best.scratch_floats = ks > 1 ? (size_t)ks * tiles * TILE_N * m * (dual ? 2 : 1) + (size_t)ks * m : 0;
        }
    }
    return best;
}

bool tc_supported(int m, int N, int K, bool dual) {
    if (m < 1 || m > CSD_MAX_ROWS || N < 1 || K < 64 || (K & 7)) return false;
    TcPlan p = tc_plan(m, N, K, dual);
    return p.grid > 0;
}

size_t tc_scratch_bytes(int m, int N, int K, bool dual) {
    size_t worst = 0;
    for (int mm = 1; mm <= m; ++mm) {
        if (!tc_supported(mm, N, K, dual)) continue;
        size_t b = tc_plan(mm, N, K, dual).scratch_floats * sizeof(float);
        if (b > worst) worst = b;
    }
    return align_up(worst, 256);
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
    const void* p; int N, K;
    bool operator==(const MapKey& o) const { return p == o.p && N == o.N && K == o.K; }
};
struct MapHash {
    size_t operator()(const MapKey& k) const { return (size_t)k.p ^ ((size_t)k.N << 20) ^ ((size_t)k.K << 40); }
};
static std::mutex g_map_mu;
static std::unordered_map<MapKey, CUtensorMap, MapHash> g_maps;

static bool weight_map(const void* W, int N, int K, CUtensorMap* out) {
    std::lock_guard<std::mutex> lk(g_map_mu);
    auto it = g_maps.find(MapKey{W, N, K});
    if (it != g_maps.end()) { *out = it->second; return true; }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    CUtensorMap tm;
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)N};
    cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    cuuint32_t box[2] = {(cuuint32_t)KB, (cuuint32_t)TILE_N};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(W), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return false;
    if (g_maps.size() > 4096) g_maps.clear();
    g_maps.emplace(MapKey{W, N, K}, tm);
    *out = tm;
    return true;
}

// ---- device-side PTX helpers -------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Bounded wait: false after SPIN_LIMIT polls.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    const uint32_t a = smem_u32(bar);
    for (int i = 0; i < SPIN_LIMIT; ++i) {
        uint32_t ok;
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                     : "=r"(ok) : "r"(a), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, uint64_t* bar, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(smem_u32(dst)), "l"((uint64_t)tm), "r"(smem_u32(bar)), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
    asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p; }"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum) : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float* v) {
    uint32_t r[16];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// K-major operand tile with 128-byte swizzle: rows of 128 bytes, 8-row atoms 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFF) >> 4);        // start address, 16-byte units
    d |= (uint64_t)1 << 16;                        // leading byte offset (unused with swizzle)
    d |= (uint64_t)(1024 >> 4) << 32;              // stride between 8-row atoms
    d |= (uint64_t)1 << 46;                        // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                        // 128-byte swizzle
    return d;
}

struct TcParams {
    const float* X; const __nv_bfloat16* gain; float* Y; float* partial; unsigned* tickets; int* status;
    int N, K, ldx, ldy, kb_per, kslices, tiles, stages, epilogue;
    float eps;
};

struct __align__(8) TcCtrl {
    uint64_t full[8], empty[8], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    int abort_flag, last_flag;
    float ss[32];
};

__device__ __forceinline__ float tc_gelu(float x) {
    return 0.5f * x * (1.f + tanhf(0.7978845608028654f * (x + 0.044715f * x * x * x)));
}
__device__ __forceinline__ float tc_silu(float x) { return x / (1.f + expf(-x)); }

template <int M, bool DUAL>
__global__ void __launch_bounds__(TC_THREADS, 1)
skinny_gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmW2,
                      const TcParams p) {
    constexpr int NPAD = 3 * M <= 16 ? 16 : (3 * M <= 32 ? 32 : (3 * M <= 48 ? 48 : 64));
    constexpr int NT = DUAL ? 2 : 1;
    constexpr int ACC_COLS = NPAD * NT;                       // tensor-memory columns per accumulator set
    constexpr int TMEM_COLS = 2 * ACC_COLS <= 32 ? 32 : (2 * ACC_COLS <= 64 ? 64 : (2 * ACC_COLS <= 128 ? 128 : 256));
    constexpr int STAGE = STAGE_BYTES * NT;
    constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NPAD >> 3) << 17) |
                               ((uint32_t)(TILE_N >> 4) << 24);   // f32 accumulate, bf16 x bf16, K-major both

    extern __shared__ unsigned char smem_raw[];
    unsigned char* base = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char* ring = base;                                            // stages x STAGE
    unsigned char* xs = ring + (size_t)p.stages * STAGE;                   // [kb_per][NPAD][128 B], swizzled
    TcCtrl* ctl = (TcCtrl*)(xs + (size_t)p.kb_per * NPAD * 128);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int ks = blockIdx.x % p.kslices;
    const int cta_in_slice = blockIdx.x / p.kslices, ctas_per_slice = gridDim.x / p.kslices;
    const int kb0 = ks * p.kb_per;
    const int nkb = min(p.kb_per, (p.K + KB - 1) / KB - kb0);            // k-blocks of this slice
    const int k0 = kb0 * KB, kw = min(p.K, k0 + nkb * KB) - k0;
    const int my_tiles = cta_in_slice < p.tiles ? (p.tiles - cta_in_slice + ctas_per_slice - 1) / ctas_per_slice : 0;
    const int items = my_tiles * nkb;

    if (tid == 0) {
        for (int s = 0; s < 8; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
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

    // item i = (local tile i / nkb, k-block i % nkb) lands in stage i % stages
    auto produce = [&](int i) {
        const int s = i % p.stages;
        const int tile = cta_in_slice + (i / nkb) * ctas_per_slice, kb = kb0 + i % nkb;
        unsigned char* dst = ring + (size_t)s * STAGE;
        mbar_expect_tx(&ctl->full[s], (uint32_t)STAGE);
        tma_load_2d(dst, &tmW, &ctl->full[s], kb * KB, tile * TILE_N);
        if (DUAL) tma_load_2d(dst + STAGE_BYTES, &tmW2, &ctl->full[s], kb * KB, tile * TILE_N);
    };
    // the weights do not depend on the kernel that produces X: fill the ring before waiting for it
    if (tid == 0)
        for (int i = 0; i < items && i < p.stages; ++i) produce(i);
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // ---- split this slice of X into three bf16 terms, rows j = term * M + r, swizzled like TMA would
    for (int i = tid; i < p.kb_per * NPAD * 8; i += TC_THREADS) reinterpret_cast<uint4*>(xs)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    {
        const int chunks = kw / 8;                         // 16-byte chunks per row (K is a multiple of 8)
        for (int r = warp; r < M; r += TC_THREADS / 32) {  // one warp per row, four chunks in flight per lane
            float sq = 0.f;
            for (int c0 = lane; c0 < chunks; c0 += 128) {
                float4 xa[4], xb[4];
                uint4 gg[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int c = c0 + 32 * u;
                    if (c < chunks) {
                        const float* src = p.X + (size_t)r * p.ldx + k0 + c * 8;
                        xa[u] = *reinterpret_cast<const float4*>(src);
                        xb[u] = *reinterpret_cast<const float4*>(src + 4);
                        if (p.gain) gg[u] = *reinterpret_cast<const uint4*>(p.gain + k0 + c * 8);
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int c = c0 + 32 * u;
                    if (c >= chunks) continue;
                    float v[8] = {xa[u].x, xa[u].y, xa[u].z, xa[u].w, xb[u].x, xb[u].y, xb[u].z, xb[u].w};
#pragma unroll
                    for (int e = 0; e < 8; ++e) sq = fmaf(v[e], v[e], sq);
                    if (p.gain) {
                        const uint4 g = gg[u];
                        v[0] *= bf16lo(g.x); v[1] *= bf16hi(g.x); v[2] *= bf16lo(g.y); v[3] *= bf16hi(g.y);
                        v[4] *= bf16lo(g.z); v[5] *= bf16hi(g.z); v[6] *= bf16lo(g.w); v[7] *= bf16hi(g.w);
                    }
                    uint32_t t1[4], t2[4], t3[4];
#pragma unroll
                    for (int e = 0; e < 8; e += 2) {
                        uint32_t w1 = 0, w2 = 0, w3 = 0;
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const float x = v[e + h];
                            const uint16_t b1 = float_to_bf16_bits(x);
                            const float r1 = x - bf16_bits_to_float(b1);
                            const uint16_t b2 = float_to_bf16_bits(r1);
                            const uint16_t b3 = float_to_bf16_bits(r1 - bf16_bits_to_float(b2));
                            w1 |= (uint32_t)b1 << (16 * h); w2 |= (uint32_t)b2 << (16 * h); w3 |= (uint32_t)b3 << (16 * h);
                        }
                        t1[e / 2] = w1; t2[e / 2] = w2; t3[e / 2] = w3;
                    }
                    const int kb = c >> 3, cc = c & 7;
                    unsigned char* blk = xs + (size_t)kb * NPAD * 128;
                    const int j1 = r, j2 = M + r, j3 = 2 * M + r;
                    *reinterpret_cast<uint4*>(blk + j1 * 128 + ((cc ^ (j1 & 7)) << 4)) = make_uint4(t1[0], t1[1], t1[2], t1[3]);
                    *reinterpret_cast<uint4*>(blk + j2 * 128 + ((cc ^ (j2 & 7)) << 4)) = make_uint4(t2[0], t2[1], t2[2], t2[3]);
                    *reinterpret_cast<uint4*>(blk + j3 * 128 + ((cc ^ (j3 & 7)) << 4)) = make_uint4(t3[0], t3[1], t3[2], t3[3]);
                }
            }
            sq = warp_sum(sq);
            if (lane == 0) ctl->ss[r] = sq;
        }
    }
    fence_async_smem();
    __syncthreads();
    float* ss_part = p.partial + (size_t)p.kslices * p.tiles * TILE_N * M * NT;   // [kslices][M]
    __syncthreads();
    if (p.kslices > 1 && p.gain) {
        if (tid < M) ss_part[ks * M + tid] = ctl->ss[tid];
        __threadfence();
        __syncthreads();
    }

    volatile int* abort_flag = &ctl->abort_flag;
    if (warp == 0) {
        // ---- TMA producer: refill a stage once the MMAs that read it have completed
        if (lane == 0) {
            for (int i = p.stages; i < items && !*abort_flag; ++i) {
                const int s = i % p.stages;
                if (!mbar_wait(&ctl->empty[s], ((i / p.stages) - 1) & 1)) { *abort_flag = 1; break; }
                produce(i);
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer
        if (lane == 0) {
            for (int t = 0; t < my_tiles && !*abort_flag; ++t) {
                const int b = t & 1;
                if (!mbar_wait(&ctl->acc_empty[b], ((t >> 1) & 1) ^ 1)) { *abort_flag = 1; break; }
                tc_fence_after();
                const uint32_t d0 = tmem + (uint32_t)(b * ACC_COLS);
                for (int kb = 0; kb < nkb; ++kb) {
                    const int i = t * nkb + kb, s = i % p.stages;
                    if (!mbar_wait(&ctl->full[s], (i / p.stages) & 1)) { *abort_flag = 1; break; }
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(ring + (size_t)s * STAGE);
                    const uint32_t b_addr = smem_u32(xs + (size_t)kb * NPAD * 128);
#pragma unroll
                    for (int k = 0; k < KB / 16; ++k) {
                        const uint64_t bd = smem_desc_sw128(b_addr + k * 32);
                        tc_mma(d0, smem_desc_sw128(a_addr + k * 32), bd, IDESC, (kb | k) != 0);
                        if (DUAL) tc_mma(d0 + NPAD, smem_desc_sw128(a_addr + STAGE_BYTES + k * 32), bd, IDESC, (kb | k) != 0);
                    }
                    tc_commit(&ctl->empty[s]);          // stage reusable once these MMAs have read it
                }
                tc_commit(&ctl->acc_full[b]);           // accumulators of this tile complete
            }
        }
    } else {
        // ---- epilogue warps: quadrant q of tensor memory holds weight rows q*32 .. q*32+31 of the tile
        const int q = warp & 3, et = (warp - 2) * 32 + lane;
        for (int t = 0; t < my_tiles; ++t) {
            const int b = t & 1, tile = cta_in_slice + t * ctas_per_slice;
            const bool ok = mbar_wait(&ctl->acc_full[b], (t >> 1) & 1);   // all four warps see the same outcome
            if (!ok) { *abort_flag = 1; break; }
            tc_fence_after();
            const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * ACC_COLS);
            float sums[NT][M];
#pragma unroll
            for (int u = 0; u < NT; ++u) {
                float third[M], second[M];
#pragma unroll
                for (int r = 0; r < M; ++r) { sums[u][r] = 0.f; second[r] = 0.f; third[r] = 0.f; }
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
                for (int r = 0; r < M; ++r) sums[u][r] += second[r] + third[r];   // small terms first
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->acc_empty[b]);
            const int n = tile * TILE_N + q * 32 + lane;
            if (p.kslices > 1) {
                float* mine = p.partial + (((size_t)ks * p.tiles + tile) * NT) * M * TILE_N;
#pragma unroll
                for (int u = 0; u < NT; ++u)
#pragma unroll
                    for (int r = 0; r < M; ++r) mine[(u * M + r) * TILE_N + q * 32 + lane] = sums[u][r];
                __threadfence();
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (et == 0) {
                    const unsigned old = atomicAdd(&p.tickets[tile], 1u);
                    ctl->last_flag = (old == (unsigned)p.kslices - 1u);
                    if (ctl->last_flag) p.tickets[tile] = 0u;
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
                const int last = ctl->last_flag;
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (!last) continue;
                __threadfence();
#pragma unroll
                for (int u = 0; u < NT; ++u)
#pragma unroll
                    for (int r = 0; r < M; ++r) {
                        float acc = 0.f;
                        for (int c = 0; c < p.kslices; ++c)
                            acc += __ldcg(p.partial + ((((size_t)c * p.tiles + tile) * NT + u) * M + r) * TILE_N + q * 32 + lane);
                        sums[u][r] = acc;
                    }
            }
            if (n < p.N) {
#pragma unroll
                for (int r = 0; r < M; ++r) {
                    float scale = 1.f;
                    if (p.gain) {
                        float sq = ctl->ss[r];
                        if (p.kslices > 1) {
                            sq = 0.f;
                            for (int c = 0; c < p.kslices; ++c) sq += __ldcg(ss_part + c * M + r);
                        }
                        scale = 1.f / sqrtf(sq / (float)p.K + p.eps);
                    }
                    float val = sums[0][r] * scale;
                    if (DUAL) {
                        const float up = sums[NT - 1][r] * scale;
                        val = (p.epilogue == EPI_GEGLU ? tc_gelu(val) : tc_silu(val)) * up;
                    }
                    float* y = p.Y + (size_t)r * p.ldy + n;
                    if (p.epilogue == EPI_ADD) *y += val; else *y = val;
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

template <int M, bool DUAL>
static csd_status launch_tc(const CUtensorMap& tw, const CUtensorMap& tw2, const TcParams& tp, const TcPlan& pl,
                            cudaStream_t st) {
    auto kern = skinny_gemm_tc_kernel<M, DUAL>;
    static bool attr_set = false;
    if (!attr_set) {
        CSD_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM_MAX + 1024));
        attr_set = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)pl.grid);
    cfg.blockDim = dim3(TC_THREADS);
    cfg.dynamicSmemBytes = pl.smem + 1024;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    CSD_CUDA(cudaLaunchKernelEx(&cfg, kern, tw, tw2, tp));
    count_launch();
    return CSD_OK;
}

csd_status launch_linear_tc(const LinearArgs& a, cudaStream_t st) {
    const bool dual = a.W2 != nullptr;
    if (!tc_supported(a.m, a.N, a.K, dual)) return CSD_ERR_UNSUPPORTED;
    if ((((uintptr_t)a.X) & 15) || (a.ldx & 3)) return CSD_ERR_INVALID_ARG;
    const TcPlan pl = tc_plan(a.m, a.N, a.K, dual);
    if (pl.kslices > 1 && (!a.partial || !a.tickets)) return CSD_ERR_INVALID_ARG;
    CUtensorMap tw, tw2;
    if (!weight_map(a.W, a.N, a.K, &tw)) return CSD_ERR_UNSUPPORTED;
    tw2 = tw;
    if (dual && !weight_map(a.W2, a.N, a.K, &tw2)) return CSD_ERR_UNSUPPORTED;
    TcParams tp;
    tp.X = a.X; tp.gain = a.gain; tp.Y = a.Y; tp.partial = a.partial; tp.tickets = a.tickets;
    tp.status = status_word_device();
    tp.N = a.N; tp.K = a.K; tp.ldx = a.ldx; tp.ldy = a.ldy; tp.kb_per = pl.kb_per; tp.kslices = pl.kslices;
    tp.tiles = pl.tiles; tp.stages = pl.stages; tp.epilogue = a.epilogue; tp.eps = a.eps;
#define CSD_TC_CASE(MM) \
    case MM: return dual ? launch_tc<MM, true>(tw, tw2, tp, pl, st) : launch_tc<MM, false>(tw, tw2, tp, pl, st);
    switch (a.m) {
        CSD_TC_CASE(1) CSD_TC_CASE(2) CSD_TC_CASE(3) CSD_TC_CASE(4) CSD_TC_CASE(5) CSD_TC_CASE(6) CSD_TC_CASE(7)
        CSD_TC_CASE(8) CSD_TC_CASE(9) CSD_TC_CASE(10) CSD_TC_CASE(11) CSD_TC_CASE(12) CSD_TC_CASE(13)
        CSD_TC_CASE(14) CSD_TC_CASE(15) CSD_TC_CASE(16) CSD_TC_CASE(17)
    }
#undef CSD_TC_CASE
    return CSD_ERR_INVALID_ARG;
}

}  // namespace csd
