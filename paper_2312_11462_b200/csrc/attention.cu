// Attention of a block of m <= 17 query rows against a bf16 K/V cache, split along the keys.
//
// grid = (heads, splits), the splits of one head forming a thread-block cluster.  A CTA walks its
// key range in tiles of 64 positions: thread 0 requests each tile's committed rows with two bulk
// copies (a head's rows are contiguous in the cache) that complete on an mbarrier, two tiles in
// flight; the block's own rows (self-attention of a drafted block) are rotated, rounded to bf16,
// written to the cache and laid over the staged tile by the CTA whose range holds them, so the
// separate append pass and its round trip through HBM are gone.  Every CTA keeps an online softmax
// per row (running max, running sum, rescaled accumulator); the splits then exchange (max, sum,
// unnormalised output) through distributed shared memory and each merges a slice of the output.
// Rows see keys [0, n_keys + r) when causal, all n_keys otherwise (cross-attention, encoder).
#include <cooperative_groups.h>
#include "attention.cuh"
#include "tc_common.cuh"

namespace cg = cooperative_groups;

namespace csd {

constexpr int AT = 256;
constexpr int TILE = 64;
constexpr int MAXM = CSD_MAX_ROWS;
constexpr int MAX_SPLITS = 8;          // portable cluster size
constexpr int STAGES = 2;

template <int DH> struct AttnCfg {
    static constexpr int HP = DH / 2;                        // dim pairs
    static constexpr int G = AT / HP;                        // row groups in the PV phase
    static constexpr int RG = (MAXM + G - 1) / G;            // rows per group
    static constexpr int NC = DH / 32;                       // 8-element chunks per score thread
    static constexpr int QROW = NC * 36;                     // q row: 32-float groups, 4 floats of skew each
    static constexpr int REC = DH + 2;                       // merge record: output row, max, sum
    static constexpr size_t TILE_BYTES = (size_t)TILE * DH * 2;
    static constexpr size_t QS_FLOATS = (size_t)MAXM * (QROW > REC ? QROW : REC);
    static constexpr size_t SMEM = 2 * STAGES * TILE_BYTES + QS_FLOATS * 4 + (size_t)MAXM * TILE * 4 +
                                   2 * (size_t)MAXM * DH * 2 + 3 * 32 * 4 + 128;
};

struct AttnParams {
    const float* q; const float* k_new; const float* v_new; const float* rope_cos; const float* rope_sin;
    __nv_bfloat16* Kc; __nv_bfloat16* Vc; const float* bias; float* out;
    __nv_bfloat16* out_xs; int out_xs_ld;
    int xs_m, xs_r0;        // three-term output: rows per term of the whole buffer, row of this block's first row
    int* status;
    int sub_rows;           // > 0: grid.z sub-blocks of this many rows each, over a cache that already holds every row
    int ldq, ld_new, m, cap, H, n_keys, n_old, early_loads, causal, bias_len, bias_zero, q_pos0, ldo, nsplit, split_len;
    float scale;
    // tree-shaped block: row r sees block row j only if bit j of tmask[r] is set (its ancestors and
    // itself) and is rotated for position n_old + tdepth[r]; its cache slot stays n_old + r
    int tree;
    unsigned tmask[MAXM];
    unsigned char tdepth[MAXM];
};

__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// two neighbouring output columns of row r as three bf16 terms each (rows term * m + r)
__device__ __forceinline__ void store_split(__nv_bfloat16* xs, int ld, int m, int r, int col, float a, float b) {
    uint16_t a1, a2, a3, c1, c2, c3;
    split3(a, a1, a2, a3);
    split3(b, c1, c2, c3);
    uint32_t* base = reinterpret_cast<uint32_t*>(reinterpret_cast<uint16_t*>(xs) + col);
    base[((size_t)r * ld) >> 1] = a1 | ((uint32_t)c1 << 16);
    base[((size_t)(m + r) * ld) >> 1] = a2 | ((uint32_t)c2 << 16);
    base[((size_t)(2 * m + r) * ld) >> 1] = a3 | ((uint32_t)c3 << 16);
}


// Merge of the splits' records (unnormalised output row, running max, running sum) through
// distributed shared memory: the CTAs of a head share out the m*DH output elements; each thread
// first fetches everything it needs from all splits in one batch of independent remote loads.
template <int DH, int REC>
__device__ __forceinline__ void merge_splits(cg::cluster_group& cluster, float* rec, const AttnParams& p, int h, int split,
                                             int m, int r0) {
    // m rows of this CTA's records; they are rows r0 .. r0+m-1 of the launch's output
    for (int i = split * AT + threadIdx.x; i < m * DH; i += p.nsplit * AT) {
        const int r = i / DH, d = i % DH;
        float ms[MAX_SPLITS], ls[MAX_SPLITS], vs[MAX_SPLITS];
#pragma unroll
        for (int s = 0; s < MAX_SPLITS; ++s) {
            ms[s] = -INFINITY; ls[s] = 0.f; vs[s] = 0.f;
            if (s < p.nsplit) {
                const float* rs = cluster.map_shared_rank(rec, s) + r * REC;
                ms[s] = rs[DH]; ls[s] = rs[DH + 1]; vs[s] = rs[d];
            }
        }
        float M = -INFINITY;
#pragma unroll
        for (int s = 0; s < MAX_SPLITS; ++s) M = fmaxf(M, ms[s]);
        float num = 0.f, den = 0.f;
#pragma unroll
        for (int s = 0; s < MAX_SPLITS; ++s)
            if (ms[s] > -INFINITY) {
                const float w = expf(ms[s] - M);
                num = fmaf(vs[s], w, num);
                den = fmaf(ls[s], w, den);
            }
        const float ov = den > 0.f ? num / den : 0.f;
        p.out[(size_t)(r0 + r) * p.ldo + h * DH + d] = ov;
        if (p.out_xs) {
            uint16_t b1, b2, b3;
            split3(ov, b1, b2, b3);
            uint16_t* xs = reinterpret_cast<uint16_t*>(p.out_xs) + h * DH + d;
            xs[(size_t)(p.xs_r0 + r0 + r) * p.out_xs_ld] = b1;
            xs[(size_t)(p.xs_m + p.xs_r0 + r0 + r) * p.out_xs_ld] = b2;
            xs[(size_t)(2 * p.xs_m + p.xs_r0 + r0 + r) * p.out_xs_ld] = b3;
        }
    }
}

template <int DH>
__global__ void __launch_bounds__(AT)
block_attention_kernel(const AttnParams p) {
    using C = AttnCfg<DH>;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __nv_bfloat16* Ks = reinterpret_cast<__nv_bfloat16*>(smem_raw);            // [STAGES][TILE][DH]
    __nv_bfloat16* Vs = Ks + STAGES * TILE * DH;
    float* qs = reinterpret_cast<float*>(Vs + STAGES * TILE * DH);            // [MAXM][QROW]; later [MAXM][REC]
    float* sc = qs + C::QS_FLOATS;                                            // [MAXM][TILE]
    __nv_bfloat16* newK = reinterpret_cast<__nv_bfloat16*>(sc + MAXM * TILE); // [MAXM][DH] the block's own rows
    __nv_bfloat16* newV = newK + MAXM * DH;
    float* row_m = reinterpret_cast<float*>(newV + MAXM * DH);                // [32]
    float* row_l = row_m + 32;
    float* row_a = row_l + 32;
    uint64_t* full = reinterpret_cast<uint64_t*>(row_a + 32);                 // [STAGES]

    cg::cluster_group cluster = cg::this_cluster();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int h = blockIdx.x, split = blockIdx.y;
    const int m = p.m, half = DH / 2;
    const int total = p.causal ? p.n_keys + m - 1 : p.n_keys;   // keys any row may see
    const int s_begin = split * p.split_len;
    const int s_end = min(total, s_begin + p.split_len);
    const int n_tiles = s_end > s_begin ? (s_end - s_begin + TILE - 1) / TILE : 0;
    __nv_bfloat16* Kh = p.Kc + (size_t)h * p.cap * DH;
    __nv_bfloat16* Vh = p.Vc + (size_t)h * p.cap * DH;
    const float* bias_h = p.bias ? p.bias + (size_t)h * p.bias_len : nullptr;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) mbar_init(&full[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 32) { row_m[tid] = -INFINITY; row_l[tid] = 0.f; row_a[tid] = 1.f; }
    __syncthreads();


    // committed rows of tile `it` (the rest of the tile, if any, are the block's own rows)
    auto old_rows = [&](int it) {
        const int t0 = s_begin + it * TILE;
        return max(0, min(min(t0 + TILE, s_end), p.n_old) - t0);
    };
    auto request = [&](int it) {
        const int st = it % STAGES, t0 = s_begin + it * TILE, cnt = old_rows(it);
        if (cnt <= 0) return;
        const uint32_t bytes = (uint32_t)cnt * DH * 2;
        mbar_expect_tx(&full[st], 2 * bytes);
        bulk_load(Ks + (size_t)st * TILE * DH, Kh + (size_t)t0 * DH, bytes, &full[st]);
        bulk_load(Vs + (size_t)st * TILE * DH, Vh + (size_t)t0 * DH, bytes, &full[st]);
    };
    // Committed rows were written by the attention kernel of an earlier forward; between that
    // kernel and this one the stream holds at least one kernel that waits for its predecessor
    // before it lets its successor start, so those rows are complete and may be requested before
    // this kernel's own dependency wait.  q and the block's k and v rows come from the kernel
    // right before this one.  The encoder's self-attention reads rows the previous kernel wrote:
    // there the requests wait too.
    if (tid == 0 && p.early_loads)
        for (int it = 0; it < n_tiles && it < STAGES; ++it) request(it);
    pdl_wait();
    pdl_trigger();
    if (tid == 0 && !p.early_loads)
        for (int it = 0; it < n_tiles && it < STAGES; ++it) request(it);

    // ---- the block's rows: q (rotated) into shared memory; k (rotated) and v rounded to bf16, kept
    //      for the tiles that hold them and written to the cache by the CTA whose range they fall in
    for (int i = tid; i < m * half; i += AT) {
        const int r = i / half, d = i % half, pos = p.n_old + r;
        const int rpos = p.n_old + (p.tree ? (int)p.tdepth[r] : r);      // position the rotation uses
        float c = 1.f, s = 0.f;
        if (p.rope_cos) { c = p.rope_cos[(size_t)rpos * half + d]; s = p.rope_sin[(size_t)rpos * half + d]; }
        const float* qr = p.q + (size_t)r * p.ldq + h * DH;
        const float q0 = qr[d], q1 = qr[d + half];
        const int e0 = d, e1 = d + half;
        qs[r * C::QROW + (e0 >> 5) * 36 + (e0 & 31)] = q0 * c - q1 * s;
        qs[r * C::QROW + (e1 >> 5) * 36 + (e1 & 31)] = q0 * s + q1 * c;
        if (p.k_new) {
            const float* kr = p.k_new + (size_t)r * p.ld_new + h * DH;
            const float* vr = p.v_new + (size_t)r * p.ld_new + h * DH;
            const float k0 = kr[d], k1 = kr[d + half];
            const __nv_bfloat16 ka = __float2bfloat16_rn(k0 * c - k1 * s), kb = __float2bfloat16_rn(k0 * s + k1 * c);
            const __nv_bfloat16 va = __float2bfloat16_rn(vr[d]), vb = __float2bfloat16_rn(vr[d + half]);
            newK[r * DH + d] = ka; newK[r * DH + d + half] = kb;
            newV[r * DH + d] = va; newV[r * DH + d + half] = vb;
            if (pos >= s_begin && pos < s_end) {
                Kh[(size_t)pos * DH + d] = ka; Kh[(size_t)pos * DH + d + half] = kb;
                Vh[(size_t)pos * DH + d] = va; Vh[(size_t)pos * DH + d + half] = vb;
            }
        }
    }

    const int dp = tid % C::HP, g = tid / C::HP;
    float acc[C::RG][2];
#pragma unroll
    for (int rr = 0; rr < C::RG; ++rr) { acc[rr][0] = 0.f; acc[rr][1] = 0.f; }

    bool failed = false;
    for (int it = 0; it < n_tiles; ++it) {
        const int st = it % STAGES, t0 = s_begin + it * TILE;
        const int ok = old_rows(it) <= 0 || mbar_wait(&full[st], (uint32_t)(it / STAGES) & 1u);
        if (__syncthreads_or(!ok)) {      // (also orders the set-up above before the first tile)
            if (!ok) mbar_wait(&full[st], (uint32_t)(it / STAGES) & 1u);   // once more, so no copy is in flight at exit
            failed = true;
            break;
        }
        __nv_bfloat16* Kt = Ks + (size_t)st * TILE * DH;
        __nv_bfloat16* Vt = Vs + (size_t)st * TILE * DH;
        const int valid = min(TILE, s_end - t0);
        {   // lay the block's own rows over the tile; clear the value rows past the end of the range
            const int new_lo = max(t0, p.n_old), n_new = t0 + valid - new_lo;
            for (int idx = tid; idx < n_new * (DH / 8); idx += AT) {
                const int row = idx / (DH / 8), c = idx % (DH / 8), j = new_lo + row - t0, r = new_lo + row - p.n_old;
                *reinterpret_cast<uint4*>(Kt + j * DH + c * 8) = *reinterpret_cast<const uint4*>(newK + r * DH + c * 8);
                *reinterpret_cast<uint4*>(Vt + j * DH + c * 8) = *reinterpret_cast<const uint4*>(newV + r * DH + c * 8);
            }
            for (int idx = tid; idx < (TILE - valid) * (DH / 8); idx += AT)
                *reinterpret_cast<uint4*>(Vt + (size_t)valid * DH + idx * 8) = make_uint4(0, 0, 0, 0);
        }
        __syncthreads();
        // ---- scores: 4 threads per key, each over a quarter of the head dimension.  The 32-element
        //      group a thread reads at step c is rotated by the key index, so that neighbouring keys
        //      (whose rows start a multiple of 128 bytes apart) hit different banks.
        {
            const int j = tid >> 2, part = tid & 3;
            uint4 kreg[C::NC];
#pragma unroll
            for (int c = 0; c < C::NC; ++c)
                kreg[c] = *reinterpret_cast<const uint4*>(Kt + j * DH + (((c + j) % C::NC) * 4 + part) * 8);
            const int key = t0 + j;
            for (int r = 0; r < m; ++r) {
                float d = 0.f;
#pragma unroll
                for (int c = 0; c < C::NC; ++c) {
                    const float* qp = qs + r * C::QROW + ((c + j) % C::NC) * 36 + part * 8;
                    const float4 qa = *reinterpret_cast<const float4*>(qp);
                    const float4 qb = *reinterpret_cast<const float4*>(qp + 4);
                    d = fmaf(bf16lo(kreg[c].x), qa.x, d); d = fmaf(bf16hi(kreg[c].x), qa.y, d);
                    d = fmaf(bf16lo(kreg[c].y), qa.z, d); d = fmaf(bf16hi(kreg[c].y), qa.w, d);
                    d = fmaf(bf16lo(kreg[c].z), qb.x, d); d = fmaf(bf16hi(kreg[c].z), qb.y, d);
                    d = fmaf(bf16lo(kreg[c].w), qb.z, d); d = fmaf(bf16hi(kreg[c].w), qb.w, d);
                }
                d += __shfl_xor_sync(0xffffffffu, d, 1);
                d += __shfl_xor_sync(0xffffffffu, d, 2);
                if (part == 0) {
                    const int limit = p.causal ? p.n_keys + r : p.n_keys;   // keys [0, limit)
                    float s = -INFINITY;
                    bool vis = key < s_end && key < limit;
                    if (p.tree && key >= p.n_old) vis = key < s_end && ((p.tmask[r] >> (key - p.n_old)) & 1u);
                    if (vis) {
                        s = d * p.scale;
                        if (bias_h) {
                            int bi = key - (p.q_pos0 + r) + p.bias_zero;
                            bi = max(0, min(p.bias_len - 1, bi));
                            s += bias_h[bi];
                        }
                    }
                    sc[r * TILE + j] = s;
                }
            }
        }
        __syncthreads();
        // ---- online softmax bookkeeping: warp w owns rows w, w+8, w+16
        for (int r = warp; r < m; r += AT / 32) {
            const float s0 = sc[r * TILE + lane], s1 = sc[r * TILE + lane + 32];
            const float tmax = warp_max(fmaxf(s0, s1));
            const float old = row_m[r];
            const float nm = fmaxf(old, tmax);
            float p0 = 0.f, p1 = 0.f, alpha = 1.f;
            if (nm > -INFINITY) {
                p0 = expf(s0 - nm);
                p1 = expf(s1 - nm);
                alpha = expf(old - nm);
            }
            sc[r * TILE + lane] = p0;
            sc[r * TILE + lane + 32] = p1;
            const float tsum = warp_sum(p0 + p1);
            if (lane == 0) {
                row_m[r] = nm;
                row_l[r] = row_l[r] * alpha + tsum;
                row_a[r] = alpha;
            }
        }
        __syncthreads();
        // ---- P.V: thread owns one dim pair for the rows of its group
#pragma unroll
        for (int rr = 0; rr < C::RG; ++rr) {
            const int r = g + rr * C::G;
            if (r < m) { const float a = row_a[r]; acc[rr][0] *= a; acc[rr][1] *= a; }
        }
        for (int j4 = 0; j4 < TILE; j4 += 4) {
            float v[4][2];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t w = *reinterpret_cast<const uint32_t*>(Vt + (j4 + i) * DH + 2 * dp);
                v[i][0] = bf16lo(w); v[i][1] = bf16hi(w);
            }
#pragma unroll
            for (int rr = 0; rr < C::RG; ++rr) {
                const int r = g + rr * C::G;
                if (r < m) {
                    const float4 pp = *reinterpret_cast<const float4*>(sc + r * TILE + j4);
                    acc[rr][0] = fmaf(pp.x, v[0][0], acc[rr][0]); acc[rr][1] = fmaf(pp.x, v[0][1], acc[rr][1]);
                    acc[rr][0] = fmaf(pp.y, v[1][0], acc[rr][0]); acc[rr][1] = fmaf(pp.y, v[1][1], acc[rr][1]);
                    acc[rr][0] = fmaf(pp.z, v[2][0], acc[rr][0]); acc[rr][1] = fmaf(pp.z, v[2][1], acc[rr][1]);
                    acc[rr][0] = fmaf(pp.w, v[3][0], acc[rr][0]); acc[rr][1] = fmaf(pp.w, v[3][1], acc[rr][1]);
                }
            }
        }
        __syncthreads();           // tile consumed: its stage may be filled again
        if (tid == 0 && it + STAGES < n_tiles) {
            fence_async_smem();    // the overlay above wrote this stage through the generic proxy
            request(it + STAGES);
        }
    }
    if (failed && tid == 0) set_status(p.status, CSD_ERR_TIMEOUT);

    if (p.nsplit == 1) {
#pragma unroll
        for (int rr = 0; rr < C::RG; ++rr) {
            const int r = g + rr * C::G;
            if (r < m) {
                const float inv = row_l[r] > 0.f ? 1.f / row_l[r] : 0.f;
                float* o = p.out + (size_t)r * p.ldo + h * DH + 2 * dp;
                o[0] = acc[rr][0] * inv; o[1] = acc[rr][1] * inv;
                if (p.out_xs) store_split(p.out_xs, p.out_xs_ld, p.xs_m, p.xs_r0 + r, h * DH + 2 * dp, o[0], o[1]);
            }
        }
        return;
    }
    // ---- leave this split's (output, max, sum) in shared memory; after the cluster barrier every
    //      CTA of the head merges its share of the output elements from all the splits' records
    float* rec = qs;      // the q rows are not needed any more (all threads are past the last tile)
#pragma unroll
    for (int rr = 0; rr < C::RG; ++rr) {
        const int r = g + rr * C::G;
        if (r < m) {
            rec[r * C::REC + 2 * dp] = acc[rr][0];
            rec[r * C::REC + 2 * dp + 1] = acc[rr][1];
        }
    }
    if (tid < m) { rec[tid * C::REC + DH] = row_m[tid]; rec[tid * C::REC + DH + 1] = row_l[tid]; }
    cluster.sync();
    merge_splits<DH, C::REC>(cluster, rec, p, h, split, m, 0);
    cluster.sync();       // no CTA leaves while another may still read its record
}

// -------------------------------------------------------------------------------------------------
// Tensor-core variant (head dimension 64 or 128): the same walk over 64-key tiles, with the two
// contractions of a tile on mma.sync (m16n8k16, bf16 operands, fp32 accumulators).  K and V tiles
// arrive by tensor-map TMA copies with the 128-byte swizzle, which makes the ldmatrix reads of
// their rows conflict-free; q and the softmax weights, fp32 quantities, enter the MMAs as a
// bf16 pair (value = hi + lo, two MMAs), so the products keep 16 mantissa bits while K and V,
// bf16 in the cache, are exact.  Warp w owns keys 8w..8w+7 of the tile in q.K^T and output
// dimensions 16w..16w+15 in P.V; rows 16..31 (a 17-row block) are a second m16 tile.
// -------------------------------------------------------------------------------------------------
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// value = hi + lo with hi = bf16(value), lo = bf16(value - hi)
__device__ __forceinline__ void split2(float v, __nv_bfloat16& hi, __nv_bfloat16& lo) {
    hi = __float2bfloat16_rn(v);
    lo = __float2bfloat16_rn(v - __bfloat162float(hi));
}

template <int DH> struct MmaCfg {
    static constexpr int QP = DH * 2 + 16;                   // bytes per q row: bf16 plus one 16-byte skew
    static constexpr int PP = TILE * 2 + 16;                 // bytes per row of softmax weights
    static constexpr int SP = TILE + 4;                      // floats per score row
    static constexpr int REC = DH + 2;
    static constexpr int NBOX = DH / 64;                     // 64-dimension (128-byte) boxes per row
    static constexpr size_t TILE_BYTES = (size_t)TILE * DH * 2;
    static constexpr size_t smem(int rows) {                 // rows = 16 or 32 operand rows
        return 1024 + 2 * STAGES * TILE_BYTES + 2 * (size_t)rows * QP + (size_t)rows * SP * 4 + 2 * (size_t)rows * PP +
               2 * (size_t)MAXM * DH * 2 + 3 * 32 * 4 + 64;
    }
};
// byte offset of 16-byte chunk c (8 dimensions) of key row j inside a swizzled tile
template <int DH> __device__ __forceinline__ uint32_t kv_off(int j, int c) {
    return (uint32_t)((c >> 3) * (TILE * 128) + j * 128 + (((c & 7) ^ (j & 7)) << 4));
}

template <int DH, int MT>
__global__ void __launch_bounds__(AT)
block_attention_mma_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                           const AttnParams p) {
    using C = MmaCfg<DH>;
    constexpr int R = MT * 16;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* base = (unsigned char*)(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
    unsigned char* Ks = base;                                        // [STAGES][tile], swizzled
    unsigned char* Vs = Ks + STAGES * C::TILE_BYTES;
    unsigned char* qh = Vs + STAGES * C::TILE_BYTES;                 // [R][QP] high parts of q; later the merge record
    unsigned char* ql = qh + R * C::QP;
    float* sc = reinterpret_cast<float*>(ql + R * C::QP);            // [R][SP]
    unsigned char* ph = reinterpret_cast<unsigned char*>(sc + R * C::SP);   // [R][PP]
    unsigned char* pl = ph + R * C::PP;
    __nv_bfloat16* newK = reinterpret_cast<__nv_bfloat16*>(pl + R * C::PP); // [MAXM][DH]
    __nv_bfloat16* newV = newK + MAXM * DH;
    float* row_m = reinterpret_cast<float*>(newV + MAXM * DH);
    float* row_l = row_m + 32;
    float* row_a = row_l + 32;
    uint64_t* full = reinterpret_cast<uint64_t*>(row_a + 32);

    cg::cluster_group cluster = cg::this_cluster();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int h = blockIdx.x, split = blockIdx.y;
    // sub-block mode (sub_rows > 0, no append): blockIdx.z picks rows r0 .. r0+m-1 of a block of p.m rows
    const int r0 = p.sub_rows ? (int)blockIdx.z * p.sub_rows : 0;
    const int m = p.sub_rows ? min(p.sub_rows, p.m - r0) : p.m, half = DH / 2;
    const int n_keys = p.n_keys + (p.causal ? r0 : 0);          // keys visible to this CTA's first row
    const int total = p.causal ? n_keys + m - 1 : n_keys;
    const int n_old = p.sub_rows ? total : p.n_old;
    const int s_begin = split * p.split_len;
    const int s_end = min(total, s_begin + p.split_len);
    const int n_tiles = s_end > s_begin ? (s_end - s_begin + TILE - 1) / TILE : 0;
    __nv_bfloat16* Kh = p.Kc + (size_t)h * p.cap * DH;
    __nv_bfloat16* Vh = p.Vc + (size_t)h * p.cap * DH;
    const float* bias_h = p.bias ? p.bias + (size_t)h * p.bias_len : nullptr;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) mbar_init(&full[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 32) { row_m[tid] = -INFINITY; row_l[tid] = 0.f; row_a[tid] = 1.f; }
    // operand rows past the block stay zero (q, and the softmax weights, which are rewritten per tile only for real rows)
    for (int i = tid; i < (2 * R * C::QP + R * C::SP * 4 + 2 * R * C::PP) / 16; i += AT)
        reinterpret_cast<uint4*>(qh)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();

    auto request = [&](int it) {       // whole 64-row boxes: rows the block itself supplies are laid over afterwards
        const int st = it % STAGES, row0 = h * p.cap + s_begin + it * TILE;
        mbar_expect_tx(&full[st], 2 * (uint32_t)C::TILE_BYTES);
#pragma unroll
        for (int b = 0; b < C::NBOX; ++b) {
            tma_load_2d(Ks + st * C::TILE_BYTES + b * (TILE * 128), &tmK, &full[st], b * 64, row0);
            tma_load_2d(Vs + st * C::TILE_BYTES + b * (TILE * 128), &tmV, &full[st], b * 64, row0);
        }
    };
    // (see the CUDA-core kernel above for why the requests may precede the dependency wait)
    if (tid == 0 && p.early_loads)
        for (int it = 0; it < n_tiles && it < STAGES; ++it) request(it);
    // this thread's (row, dimension pair) items of the block; their rotation factors are constants
    constexpr int ITEMS = ((R < MAXM ? R : (MT == 2 ? R : MAXM)) * (DH / 2) + AT - 1) / AT;
    float rc[ITEMS], rs[ITEMS];
#pragma unroll
    for (int e = 0; e < ITEMS; ++e) {
        const int i = tid + e * AT;
        rc[e] = 1.f; rs[e] = 0.f;
        if (i < m * half && p.rope_cos) {
            const size_t at = (size_t)(n_old + (p.tree ? (int)p.tdepth[i / half] : i / half)) * half + i % half;
            rc[e] = p.rope_cos[at]; rs[e] = p.rope_sin[at];
        }
    }
    pdl_wait();
    pdl_trigger();
    if (tid == 0 && !p.early_loads)
        for (int it = 0; it < n_tiles && it < STAGES; ++it) request(it);

    // ---- the block's rows: q rotated and split into its bf16 pair; k rotated, v, both rounded to bf16.
    //      All loads first (one round trip), then the arithmetic and the stores.
    {
        float qv[ITEMS][2], kv[ITEMS][2], vv[ITEMS][2];
#pragma unroll
        for (int e = 0; e < ITEMS; ++e) {
            const int i = tid + e * AT;
            if (i < m * half) {
                const int r = i / half, d = i % half;
                const float* qr = p.q + (size_t)(r0 + r) * p.ldq + h * DH;
                qv[e][0] = qr[d]; qv[e][1] = qr[d + half];
                if (p.k_new) {
                    const float* kr = p.k_new + (size_t)r * p.ld_new + h * DH;
                    const float* vr = p.v_new + (size_t)r * p.ld_new + h * DH;
                    kv[e][0] = kr[d]; kv[e][1] = kr[d + half];
                    vv[e][0] = vr[d]; vv[e][1] = vr[d + half];
                }
            }
        }
#pragma unroll
        for (int e = 0; e < ITEMS; ++e) {
            const int i = tid + e * AT;
            if (i < m * half) {
                const int r = i / half, d = i % half, pos = n_old + r;
                const float c = rc[e], s = rs[e];
                __nv_bfloat16 h0, l0, h1, l1;
                split2(qv[e][0] * c - qv[e][1] * s, h0, l0);
                split2(qv[e][0] * s + qv[e][1] * c, h1, l1);
                __nv_bfloat16* qhr = reinterpret_cast<__nv_bfloat16*>(qh + r * C::QP);
                __nv_bfloat16* qlr = reinterpret_cast<__nv_bfloat16*>(ql + r * C::QP);
                qhr[d] = h0; qhr[d + half] = h1; qlr[d] = l0; qlr[d + half] = l1;
                if (p.k_new) {
                    const __nv_bfloat16 ka = __float2bfloat16_rn(kv[e][0] * c - kv[e][1] * s);
                    const __nv_bfloat16 kb = __float2bfloat16_rn(kv[e][0] * s + kv[e][1] * c);
                    const __nv_bfloat16 va = __float2bfloat16_rn(vv[e][0]), vb = __float2bfloat16_rn(vv[e][1]);
                    newK[r * DH + d] = ka; newK[r * DH + d + half] = kb;
                    newV[r * DH + d] = va; newV[r * DH + d + half] = vb;
                    if (pos >= s_begin && pos < s_end) {
                        Kh[(size_t)pos * DH + d] = ka; Kh[(size_t)pos * DH + d + half] = kb;
                        Vh[(size_t)pos * DH + d] = va; Vh[(size_t)pos * DH + d + half] = vb;
                    }
                }
            }
        }
    }

    float o[MT][2][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int t = 0; t < 2; ++t)
#pragma unroll
            for (int e = 0; e < 4; ++e) o[mt][t][e] = 0.f;
    const int lrow = lane & 7, lmat = lane >> 3;          // ldmatrix: this lane addresses row lrow of matrix lmat
    const uint32_t qh_s = smem_u32(qh), ql_s = smem_u32(ql), ph_s = smem_u32(ph), pl_s = smem_u32(pl);

    // The q operand is the same for every tile: each warp keeps the A fragments of its row tile in
    // registers (high parts; the low parts too while a block is one row tile) instead of fetching
    // them from shared memory per tile, which is what bounded the score step.  A warp takes the row
    // tile mtw and MT groups of 8 keys of every tile.
    constexpr bool QLO_REG = MT == 1;
    const int mtw = MT == 1 ? 0 : warp >> 2;
    const int key0 = MT == 1 ? 8 * warp : 16 * (warp & 3);
    uint32_t qfh[DH / 16][4], qfl[QLO_REG ? DH / 16 : 1][4];
    __syncthreads();                        // the block's q rows are in shared memory
#pragma unroll
    for (int ks = 0; ks < DH / 16; ++ks) {
        const uint32_t aoff = (uint32_t)((mtw * 16 + (lmat & 1) * 8 + lrow) * C::QP + (2 * ks + (lmat >> 1)) * 16);
        ldsm_x4(qh_s + aoff, qfh[ks]);
        if (QLO_REG) ldsm_x4(ql_s + aoff, qfl[QLO_REG ? ks : 0]);
    }

    float run_m[R / 8], run_l[R / 8];       // running maximum and this lane's share of the running sum, rows warp + 8 i
#pragma unroll
    for (int i = 0; i < R / 8; ++i) { run_m[i] = -INFINITY; run_l[i] = 0.f; }
    bool failed = false;
    for (int it = 0; it < n_tiles; ++it) {
        const int st = it % STAGES, t0 = s_begin + it * TILE;
        const int ok = mbar_wait(&full[st], (uint32_t)(it / STAGES) & 1u);
        if (__syncthreads_or(!ok)) {
            if (!ok) mbar_wait(&full[st], (uint32_t)(it / STAGES) & 1u);
            failed = true;
            break;
        }
        // every thread is past the previous tile (the barrier above): its stage may be filled again
        if (tid == 0 && it >= 1 && it - 1 + STAGES < n_tiles) {
            fence_async_smem();
            request(it - 1 + STAGES);
        }
        unsigned char* Kt = Ks + st * C::TILE_BYTES;
        unsigned char* Vt = Vs + st * C::TILE_BYTES;
        const int valid = min(TILE, s_end - t0);
        const int new_lo = max(t0, n_old), n_new = t0 + valid - new_lo;
        if (n_new > 0 || valid < TILE) {       // same for every thread
            for (int idx = tid; idx < n_new * (DH / 8); idx += AT) {
                const int row = idx / (DH / 8), c = idx % (DH / 8), j = new_lo + row - t0, r = new_lo + row - n_old;
                *reinterpret_cast<uint4*>(Kt + kv_off<DH>(j, c)) = *reinterpret_cast<const uint4*>(newK + r * DH + c * 8);
                *reinterpret_cast<uint4*>(Vt + kv_off<DH>(j, c)) = *reinterpret_cast<const uint4*>(newV + r * DH + c * 8);
            }
            for (int idx = tid; idx < (TILE - valid) * (DH / 8); idx += AT) {
                const int j = valid + idx / (DH / 8), c = idx % (DH / 8);
                *reinterpret_cast<uint4*>(Vt + kv_off<DH>(j, c)) = make_uint4(0, 0, 0, 0);
            }
            __syncthreads();
        }
        // ---- scores of this warp's row tile against its MT groups of 8 keys; the high and low parts of q and
        //      the two halves of the head dimension accumulate separately, so that no chain is longer than DH/32 MMAs
        {
            float sacc2[MT][2][2][4];           // [key group][q part][half of the k steps]
#pragma unroll
            for (int g = 0; g < MT; ++g)
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    sacc2[g][0][0][e] = sacc2[g][0][1][e] = sacc2[g][1][0][e] = sacc2[g][1][1][e] = 0.f;
            const uint32_t Kt_s = smem_u32(Kt);
#pragma unroll
            for (int ks2 = 0; ks2 < DH / 32; ++ks2) {
#pragma unroll
                for (int g = 0; g < MT; ++g) {
                    uint32_t kb[4];
                    ldsm_x4(Kt_s + kv_off<DH>(key0 + 8 * g + lrow, 4 * ks2 + lmat), kb);
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf) {
                        const int ks = 2 * ks2 + hf;
                        mma_bf16(sacc2[g][0][hf], qfh[ks], kb[2 * hf], kb[2 * hf + 1]);
                        if (QLO_REG) {
                            mma_bf16(sacc2[g][1][hf], qfl[QLO_REG ? ks : 0], kb[2 * hf], kb[2 * hf + 1]);
                        } else {
                            const uint32_t aoff = (uint32_t)((mtw * 16 + (lmat & 1) * 8 + lrow) * C::QP + (2 * ks + (lmat >> 1)) * 16);
                            uint32_t a[4];
                            ldsm_x4(ql_s + aoff, a);
                            mma_bf16(sacc2[g][1][hf], a, kb[2 * hf], kb[2 * hf + 1]);
                        }
                    }
                }
            }
#pragma unroll
            for (int g = 0; g < MT; ++g)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int r = mtw * 16 + (lane >> 2) + (e >> 1) * 8, j = key0 + 8 * g + (lane & 3) * 2 + (e & 1);
                    if (r < m) {
                        const int key = t0 + j, limit = p.causal ? n_keys + r : n_keys;
                        float s = -INFINITY;
                        bool vis = key < s_end && key < limit;
                        if (p.tree && key >= n_old) vis = key < s_end && ((p.tmask[r] >> (key - n_old)) & 1u);
                        if (vis) {
                            s = ((sacc2[g][1][0][e] + sacc2[g][1][1][e]) + (sacc2[g][0][0][e] + sacc2[g][0][1][e])) * p.scale;
                            if (bias_h) {
                                int bi = key - (p.q_pos0 + r0 + r) + p.bias_zero;
                                bi = max(0, min(p.bias_len - 1, bi));
                                s += bias_h[bi];
                            }
                        }
                        sc[r * C::SP + j] = s;
                    }
                }
        }
        __syncthreads();
        // ---- online softmax: warp w owns rows w, w+8, ...; the weights leave as bf16 pairs.  The rows of a
        //      warp are independent, so their loads, shuffles and exponentials interleave; the row sums stay
        //      as per-lane partial sums until the walk is over.
        {
            float s0[R / 8], s1[R / 8], tmax[R / 8];
#pragma unroll
            for (int i = 0; i < R / 8; ++i) {
                const int r = warp + 8 * i;
                s0[i] = s1[i] = -INFINITY;
                if (r < m) { s0[i] = sc[r * C::SP + lane]; s1[i] = sc[r * C::SP + lane + 32]; }
                tmax[i] = fmaxf(s0[i], s1[i]);
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1)
#pragma unroll
                for (int i = 0; i < R / 8; ++i) tmax[i] = fmaxf(tmax[i], __shfl_xor_sync(0xffffffffu, tmax[i], off));
#pragma unroll
            for (int i = 0; i < R / 8; ++i) {
                const int r = warp + 8 * i;
                if (r >= m) continue;
                const float old = run_m[i];
                const float nm = fmaxf(old, tmax[i]);
                float p0 = 0.f, p1 = 0.f, alpha = 1.f;
                if (nm > -INFINITY) {
                    p0 = expf(s0[i] - nm);
                    p1 = expf(s1[i] - nm);
                    alpha = expf(old - nm);
                }
                __nv_bfloat16 h0, l0, h1, l1;
                split2(p0, h0, l0);
                split2(p1, h1, l1);
                __nv_bfloat16* phr = reinterpret_cast<__nv_bfloat16*>(ph + r * C::PP);
                __nv_bfloat16* plr = reinterpret_cast<__nv_bfloat16*>(pl + r * C::PP);
                phr[lane] = h0; phr[lane + 32] = h1; plr[lane] = l0; plr[lane + 32] = l1;
                // the sum runs over the weights as the MMA will see them
                run_l[i] = run_l[i] * alpha + ((__bfloat162float(h0) + __bfloat162float(l0)) + (__bfloat162float(h1) + __bfloat162float(l1)));
                run_m[i] = nm;
                if (lane == 0) row_a[r] = alpha;
            }
        }
        __syncthreads();
        // ---- P.V for output dimensions 16*warp .. 16*warp+15
        if (warp < DH / 16) {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                const float a0 = row_a[mt * 16 + (lane >> 2)], a1 = row_a[mt * 16 + (lane >> 2) + 8];
#pragma unroll
                for (int t = 0; t < 2; ++t) { o[mt][t][0] *= a0; o[mt][t][1] *= a0; o[mt][t][2] *= a1; o[mt][t][3] *= a1; }
            }
            const uint32_t Vt_s = smem_u32(Vt);
            float ol[MT][2][4];                 // the low parts of the weights accumulate on their own chain
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int t = 0; t < 2; ++t)
#pragma unroll
                    for (int e = 0; e < 4; ++e) ol[mt][t][e] = 0.f;
#pragma unroll
            for (int ks = 0; ks < TILE / 16; ++ks) {
                uint32_t vb[4];
                ldsm_x4_t(Vt_s + kv_off<DH>(16 * ks + (lmat & 1) * 8 + lrow, 2 * warp + (lmat >> 1)), vb);
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    const uint32_t aoff = (uint32_t)((mt * 16 + (lmat & 1) * 8 + lrow) * C::PP + (2 * ks + (lmat >> 1)) * 16);
                    uint32_t a[4];
                    ldsm_x4(ph_s + aoff, a);
                    mma_bf16(o[mt][0], a, vb[0], vb[1]);
                    mma_bf16(o[mt][1], a, vb[2], vb[3]);
                    ldsm_x4(pl_s + aoff, a);
                    mma_bf16(ol[mt][0], a, vb[0], vb[1]);
                    mma_bf16(ol[mt][1], a, vb[2], vb[3]);
                }
            }
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int t = 0; t < 2; ++t)
#pragma unroll
                    for (int e = 0; e < 4; ++e) o[mt][t][e] += ol[mt][t][e];
        }
    }
    if (failed && tid == 0) set_status(p.status, CSD_ERR_TIMEOUT);
#pragma unroll
    for (int i = 0; i < R / 8; ++i) {
        const float l = warp_sum(run_l[i]);
        const int r = warp + 8 * i;
        if (lane == 0 && r < m) { row_m[r] = run_m[i]; row_l[r] = l; }
    }
    __syncthreads();


    // element (mt, t, e) of `o`: row mt*16 + lane/4 (+8 for e >= 2), dimension 16*warp + 8*t + 2*(lane%4) + (e&1)
    if (p.nsplit == 1) {
        if (warp < DH / 16) {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int hr = 0; hr < 2; ++hr) {
                    const int r = mt * 16 + (lane >> 2) + hr * 8;
                    if (r >= m) continue;
                    const float inv = row_l[r] > 0.f ? 1.f / row_l[r] : 0.f;
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        const int d = 16 * warp + 8 * t + 2 * (lane & 3);
                        float* dst = p.out + (size_t)(r0 + r) * p.ldo + h * DH + d;
                        dst[0] = o[mt][t][2 * hr] * inv; dst[1] = o[mt][t][2 * hr + 1] * inv;
                        if (p.out_xs) store_split(p.out_xs, p.out_xs_ld, p.xs_m, p.xs_r0 + r0 + r, h * DH + d, dst[0], dst[1]);
                    }
                }
        }
        return;
    }
    float* rec = reinterpret_cast<float*>(qh);      // q is not needed any more (all threads are past the last tile)
    if (warp < DH / 16) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int hr = 0; hr < 2; ++hr) {
                const int r = mt * 16 + (lane >> 2) + hr * 8;
                if (r >= m) continue;
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    const int d = 16 * warp + 8 * t + 2 * (lane & 3);
                    rec[r * C::REC + d] = o[mt][t][2 * hr];
                    rec[r * C::REC + d + 1] = o[mt][t][2 * hr + 1];
                }
            }
    }
    if (tid < m) { rec[tid * C::REC + DH] = row_m[tid]; rec[tid * C::REC + DH + 1] = row_l[tid]; }
    cluster.sync();
    merge_splits<DH, C::REC>(cluster, rec, p, h, split, m, r0);
    cluster.sync();       // no CTA leaves while another may still read its record
}
// One 64-key tile per CTA while that keeps the splits of a head inside one portable cluster (8)
// and the grid near two CTAs per SM: short caches are latency-bound, and more splits mean more
// tiles in flight at once; long caches walk several tiles per CTA, two requests ahead.
static bool g_attn_cuda_cores = false;
void set_attention_cuda_cores(bool on) { g_attn_cuda_cores = on; }

int attn_splits(int total_keys, int H) {
    int by_sm = (2 * 148 + H - 1) / H;
    int by_len = (total_keys + TILE - 1) / TILE;
    int n = by_sm < by_len ? by_sm : by_len;
    if (n < 1) n = 1;
    if (n > MAX_SPLITS) n = MAX_SPLITS;
    return n;
}

static void attn_launch_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute* attr, const AttnParams& ap, size_t smem,
                               cudaStream_t st) {
    cfg = cudaLaunchConfig_t{};
    cfg.gridDim = dim3((unsigned)ap.H, (unsigned)ap.nsplit,
                       (unsigned)(ap.sub_rows > 0 ? (ap.m + ap.sub_rows - 1) / ap.sub_rows : 1));
    cfg.blockDim = dim3(AT);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;      // the splits of one head exchange results on chip
    attr[1].val.clusterDim.x = 1; attr[1].val.clusterDim.y = (unsigned)ap.nsplit; attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
}

template <int DH>
static csd_status launch_dh(const AttnParams& ap, cudaStream_t st) {
    auto kern = block_attention_kernel<DH>;
    static bool attr_set = false;
    if (!attr_set) {
        CSD_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AttnCfg<DH>::SMEM));
        attr_set = true;
    }
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    attn_launch_config(cfg, attr, ap, AttnCfg<DH>::SMEM, st);
    CSD_CUDA(cudaLaunchKernelEx(&cfg, kern, ap));
    count_launch();
    return CSD_OK;
}

template <int DH, int MT>
static csd_status launch_mma(const CUtensorMap& tk, const CUtensorMap& tv, const AttnParams& ap, cudaStream_t st) {
    auto kern = block_attention_mma_kernel<DH, MT>;
    static bool attr_set = false;
    const size_t smem = MmaCfg<DH>::smem(MT * 16);
    if (!attr_set) {
        CSD_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr_set = true;
    }
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    attn_launch_config(cfg, attr, ap, smem, st);
    CSD_CUDA(cudaLaunchKernelEx(&cfg, kern, tk, tv, ap));
    count_launch();
    return CSD_OK;
}

// Blocks of more than MAXM rows over a cache that already holds their keys (wide prefill, encoder):
// one launch whose grid.z walks sub-blocks of 32 rows on the tensor-core kernel; elsewhere one
// launch per MAXM rows.
static csd_status launch_attention_rows(const AttnArgs& a, cudaStream_t st);
static csd_status launch_attention_block(const AttnArgs& a, int sub_rows, cudaStream_t st);

csd_status launch_attention(const AttnArgs& a, cudaStream_t st) {
    if (a.m > MAXM) return launch_attention_rows(a, st);
    return launch_attention_block(a, 0, st);
}

static csd_status launch_attention_rows(const AttnArgs& a, cudaStream_t st) {
    if (a.k_new || a.tree_mask || a.out_xs || a.m > 128) return CSD_ERR_INVALID_ARG;   // 128: the widest block the model driver forms
    if ((a.Dh == 64 || a.Dh == 128) && !g_attn_cuda_cores) return launch_attention_block(a, 32, st);
    for (int r0 = 0; r0 < a.m; r0 += MAXM) {
        AttnArgs s = a;
        s.q = a.q + (size_t)r0 * a.ldq; s.m = a.m - r0 < MAXM ? a.m - r0 : MAXM;
        s.n_keys = a.causal ? a.n_keys + r0 : a.n_keys;
        s.q_pos0 = a.q_pos0 + r0;
        s.out = a.out + (size_t)r0 * a.ldo;
        const csd_status rc = launch_attention_block(s, 0, st);
        if (rc != CSD_OK) return rc;
    }
    return CSD_OK;
}

static csd_status launch_attention_block(const AttnArgs& a, int sub_rows, cudaStream_t st) {
    if (!a.q || !a.Kc || !a.Vc || !a.out || a.m < 1 || (sub_rows == 0 && a.m > MAXM) || a.H < 1 || a.n_keys < 0)
        return CSD_ERR_INVALID_ARG;
    const bool append = a.k_new != nullptr;
    if (append && (!a.v_new || !a.causal || a.n_keys < 1)) return CSD_ERR_INVALID_ARG;
    if ((a.rope_cos != nullptr) != (a.rope_sin != nullptr) || (a.rope_cos && !append)) return CSD_ERR_INVALID_ARG;
    if ((((uintptr_t)a.Kc) & 15) || (((uintptr_t)a.Vc) & 15)) return CSD_ERR_INVALID_ARG;
    const int total = a.causal ? a.n_keys + a.m - 1 : a.n_keys;
    if (total < 1 || total > a.cap) return CSD_ERR_CAPACITY;
    AttnParams ap;
    ap.q = a.q; ap.k_new = a.k_new; ap.v_new = a.v_new; ap.ld_new = a.ld_new; ap.rope_cos = a.rope_cos;
    ap.rope_sin = a.rope_sin; ap.Kc = a.Kc; ap.Vc = a.Vc; ap.bias = a.bias; ap.out = a.out;
    ap.status = status_word_device();
    ap.ldq = a.ldq; ap.m = a.m; ap.cap = a.cap; ap.H = a.H; ap.n_keys = a.n_keys;
    ap.n_old = append ? a.n_keys - 1 : total;
    ap.early_loads = a.kv_settled ? 1 : 0;
    ap.causal = a.causal; ap.bias_len = a.bias_len; ap.bias_zero = a.bias_zero; ap.q_pos0 = a.q_pos0;
    ap.ldo = a.ldo; ap.scale = a.scale; ap.out_xs = a.out_xs; ap.out_xs_ld = a.out_xs_ld;
    ap.xs_m = a.out_xs_rows > 0 ? a.out_xs_rows : a.m; ap.xs_r0 = a.out_xs_row0;
    ap.tree = 0;
    if (a.tree_mask) {
        if (!append || !a.tree_depth || a.bias) return CSD_ERR_INVALID_ARG;
        ap.tree = 1;
        for (int r = 0; r < MAXM; ++r) { ap.tmask[r] = r < a.m ? a.tree_mask[r] : 0u; ap.tdepth[r] = r < a.m ? (unsigned char)a.tree_depth[r] : 0; }
    }
    ap.sub_rows = sub_rows;
    // sub-blocks: each (head, sub-block) pair is a cluster of its own; the split length follows the
    // last sub-block, which sees the most keys (earlier ones leave their last splits empty)
    ap.nsplit = attn_splits(total, sub_rows > 0 ? a.H * ((a.m + sub_rows - 1) / sub_rows) : a.H);
    if (sub_rows > 0) {
        // these launches are throughput-bound: as many splits as keep the whole grid resident at once
        // (two CTAs per SM), rather than one more that spills into a second wave
        const int pairs = a.H * ((a.m + sub_rows - 1) / sub_rows);
        int fit = 2 * 148 / pairs;
        if (fit < 1) fit = 1;
        if (ap.nsplit > fit) ap.nsplit = fit;
    }
    int len = (total + ap.nsplit - 1) / ap.nsplit;
    ap.split_len = (len + TILE - 1) / TILE * TILE;
    ap.nsplit = (total + ap.split_len - 1) / ap.split_len;
    // head dimensions 64 and 128 run on the tensor cores; the caches then need tensor maps (rows = all heads' positions)
    if ((a.Dh == 64 || a.Dh == 128) && !g_attn_cuda_cores) {
        CUtensorMap tk, tv;
        if (tensor_map_2d(a.Kc, a.H * a.cap, a.Dh, TILE, &tk) && tensor_map_2d(a.Vc, a.H * a.cap, a.Dh, TILE, &tv)) {
            const bool one_tile = sub_rows == 0 && a.m <= 16;
            if (a.Dh == 64) return one_tile ? launch_mma<64, 1>(tk, tv, ap, st) : launch_mma<64, 2>(tk, tv, ap, st);
            return one_tile ? launch_mma<128, 1>(tk, tv, ap, st) : launch_mma<128, 2>(tk, tv, ap, st);
        }
    }
    if (sub_rows > 0) return CSD_ERR_UNSUPPORTED;     // sub-blocks exist on the tensor-core kernel only
    switch (a.Dh) {
        case 32: return launch_dh<32>(ap, st);
        case 64: return launch_dh<64>(ap, st);
        case 128: return launch_dh<128>(ap, st);
    }
    return CSD_ERR_SHAPE;
}

}  // namespace csd

extern "C" csd_status csd_set_attention_path(int path) {
    if (path < 0 || path > 1) return CSD_ERR_INVALID_ARG;
    csd::set_attention_cuda_cores(path == 1);
    return CSD_OK;
}
