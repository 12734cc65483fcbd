// Attention of a block of m <= 17 query rows against a bf16 K/V cache, split along the keys.
//
// grid = (heads, splits).  A CTA walks its key range in tiles of 64 positions staged in shared
// memory, keeps an online softmax per row (running max, running sum, rescaled accumulator) and
// leaves (max, sum, unnormalised output) in scratch; the CTA that arrives last at the head's
// ticket merges the splits.  Rows see keys [0, n_keys + r] when causal (the drafted block is
// causal inside itself), all n_keys otherwise (cross-attention, encoder).
#include "attention.cuh"

namespace csd {

constexpr int AT = 256;
constexpr int TILE = 64;
constexpr int MAXM = CSD_MAX_ROWS;
constexpr int MAX_SPLITS = 32;

template <int DH> struct AttnCfg {
    static constexpr int KROW = DH + (DH == 32 ? 0 : 32);   // bf16 elements per staged row (bank spread)
    static constexpr int HP = DH / 2;                        // dim pairs
    static constexpr int G = AT / HP;                        // row groups in the PV phase
    static constexpr int RG = (MAXM + G - 1) / G;            // rows per group
    static constexpr int NC = DH / 32;                       // 8-element chunks per score thread
    static constexpr size_t SMEM = (size_t)2 * TILE * KROW * 2 + (size_t)MAXM * DH * 4 + (size_t)MAXM * TILE * 4 +
                                   3 * 32 * 4;
};

struct AttnParams {
    const float* q; const __nv_bfloat16* Kc; const __nv_bfloat16* Vc; const float* bias; float* out;
    __nv_bfloat16* out_xs; int out_xs_ld;
    float* partial; unsigned* tickets;
    int ldq, m, cap, H, n_keys, causal, bias_len, bias_zero, q_pos0, ldo, nsplit, split_len;
    float scale;
};

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

template <int DH>
__global__ void __launch_bounds__(AT)
block_attention_kernel(const AttnParams p) {
    using C = AttnCfg<DH>;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __nv_bfloat16* Ks = reinterpret_cast<__nv_bfloat16*>(smem_raw);
    __nv_bfloat16* Vs = Ks + TILE * C::KROW;
    float* qs = reinterpret_cast<float*>(Vs + TILE * C::KROW);   // [MAXM][DH]
    float* sc = qs + MAXM * DH;                                  // [MAXM][TILE]
    float* row_m = sc + MAXM * TILE;                             // [32]
    float* row_l = row_m + 32;
    float* row_a = row_l + 32;
    __shared__ int s_last;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int h = blockIdx.x, split = blockIdx.y;
    const int m = p.m;
    const int total = p.causal ? p.n_keys + m - 1 : p.n_keys;   // keys any row may see
    const int s_begin = split * p.split_len;
    const int s_end = min(total, s_begin + p.split_len);

    pdl_wait();       // q and the appended K/V rows come from the kernels before this one
    pdl_trigger();
    for (int i = tid; i < m * DH; i += AT) qs[i] = p.q[(size_t)(i / DH) * p.ldq + h * DH + (i % DH)];
    if (tid < 32) { row_m[tid] = -INFINITY; row_l[tid] = 0.f; row_a[tid] = 1.f; }

    const int dp = tid % C::HP, g = tid / C::HP;
    float acc[C::RG][2];
#pragma unroll
    for (int rr = 0; rr < C::RG; ++rr) { acc[rr][0] = 0.f; acc[rr][1] = 0.f; }

    const __nv_bfloat16* Kh = p.Kc + (size_t)h * p.cap * DH;
    const __nv_bfloat16* Vh = p.Vc + (size_t)h * p.cap * DH;
    const float* bias_h = p.bias ? p.bias + (size_t)h * p.bias_len : nullptr;

    for (int t0 = s_begin; t0 < s_end; t0 += TILE) {
        __syncthreads();   // previous tile fully consumed (also orders the qs / row state set-up)
        for (int idx = tid; idx < TILE * (DH / 8); idx += AT) {
            const int j = idx / (DH / 8), c = idx % (DH / 8);
            uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
            if (t0 + j < s_end) {
                kv = *reinterpret_cast<const uint4*>(Kh + (size_t)(t0 + j) * DH + c * 8);
                vv = *reinterpret_cast<const uint4*>(Vh + (size_t)(t0 + j) * DH + c * 8);
            }
            *reinterpret_cast<uint4*>(Ks + j * C::KROW + c * 8) = kv;
            *reinterpret_cast<uint4*>(Vs + j * C::KROW + c * 8) = vv;
        }
        __syncthreads();
        // ---- scores: 4 threads per key, each over a quarter of the head dimension
        {
            const int j = tid >> 2, part = tid & 3;
            uint4 kreg[C::NC];
#pragma unroll
            for (int c = 0; c < C::NC; ++c)
                kreg[c] = *reinterpret_cast<const uint4*>(Ks + j * C::KROW + (c * 4 + part) * 8);
            const int key = t0 + j;
            for (int r = 0; r < m; ++r) {
                float d = 0.f;
#pragma unroll
                for (int c = 0; c < C::NC; ++c) {
                    const float* qp = qs + r * DH + (c * 4 + part) * 8;
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
                    if (key < s_end && key < limit) {
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
                const uint32_t w = *reinterpret_cast<const uint32_t*>(Vs + (j4 + i) * C::KROW + 2 * dp);
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
    }
    __syncthreads();

    if (p.nsplit == 1) {
#pragma unroll
        for (int rr = 0; rr < C::RG; ++rr) {
            const int r = g + rr * C::G;
            if (r < m) {
                const float inv = row_l[r] > 0.f ? 1.f / row_l[r] : 0.f;
                float* o = p.out + (size_t)r * p.ldo + h * DH + 2 * dp;
                o[0] = acc[rr][0] * inv; o[1] = acc[rr][1] * inv;
                if (p.out_xs) store_split(p.out_xs, p.out_xs_ld, m, r, h * DH + 2 * dp, o[0], o[1]);
            }
        }
        return;
    }
    // ---- leave this split's partial result, last arrival merges
    constexpr int REC = DH + 2;
    float* mine = p.partial + ((size_t)h * p.nsplit + split) * MAXM * REC;
#pragma unroll
    for (int rr = 0; rr < C::RG; ++rr) {
        const int r = g + rr * C::G;
        if (r < m) {
            mine[r * REC + 2 * dp] = acc[rr][0];
            mine[r * REC + 2 * dp + 1] = acc[rr][1];
        }
    }
    if (tid < m) { mine[tid * REC + DH] = row_m[tid]; mine[tid * REC + DH + 1] = row_l[tid]; }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        unsigned old = atomicAdd(&p.tickets[h], 1u);
        s_last = (old == (unsigned)p.nsplit - 1u);
        if (s_last) p.tickets[h] = 0u;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const float* all = p.partial + (size_t)h * p.nsplit * MAXM * REC;
    for (int i = tid; i < m * DH; i += AT) {
        const int r = i / DH, d = i % DH;
        float M = -INFINITY;
        for (int s = 0; s < p.nsplit; ++s) M = fmaxf(M, __ldcg(all + ((size_t)s * MAXM + r) * REC + DH));
        float num = 0.f, den = 0.f;
        for (int s = 0; s < p.nsplit; ++s) {
            const float* rec = all + ((size_t)s * MAXM + r) * REC;
            const float ms = __ldcg(rec + DH);
            if (ms > -INFINITY) {
                const float w = expf(ms - M);
                num = fmaf(__ldcg(rec + d), w, num);
                den = fmaf(__ldcg(rec + DH + 1), w, den);
            }
        }
        const float o = den > 0.f ? num / den : 0.f;
        p.out[(size_t)r * p.ldo + h * DH + d] = o;
        if (p.out_xs) {
            uint16_t b1, b2, b3;
            split3(o, b1, b2, b3);
            uint16_t* xs = reinterpret_cast<uint16_t*>(p.out_xs) + h * DH + d;
            xs[(size_t)r * p.out_xs_ld] = b1;
            xs[(size_t)(m + r) * p.out_xs_ld] = b2;
            xs[(size_t)(2 * m + r) * p.out_xs_ld] = b3;
        }
    }
}

// One 64-key tile per CTA while that still gives no more than about two CTAs per SM: short caches
// are latency-bound, and a CTA that walks several tiles pays one round trip per tile.
int attn_splits(int total_keys, int H) {
    int by_sm = (2 * 148 + H - 1) / H;
    int by_len = (total_keys + TILE - 1) / TILE;
    int n = by_sm < by_len ? by_sm : by_len;
    if (n < 1) n = 1;
    if (n > MAX_SPLITS) n = MAX_SPLITS;
    return n;
}

size_t attn_scratch_bytes(int max_keys, int H, int Dh) {
    (void)max_keys;
    return align_up((size_t)H * MAX_SPLITS * MAXM * (Dh + 2) * sizeof(float), 256);
}

template <int DH>
static csd_status launch_dh(const AttnParams& ap, cudaStream_t st) {
    auto kern = block_attention_kernel<DH>;
    static bool attr_set = false;
    if (!attr_set) {
        CSD_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AttnCfg<DH>::SMEM));
        attr_set = true;
    }
    PdlLaunch L(dim3((unsigned)ap.H, (unsigned)ap.nsplit), dim3(AT), AttnCfg<DH>::SMEM, st);
    CSD_CUDA(cudaLaunchKernelEx(&L.cfg, kern, ap));
    count_launch();
    return CSD_OK;
}

csd_status launch_attention(const AttnArgs& a, cudaStream_t st) {
    if (!a.q || !a.Kc || !a.Vc || !a.out || a.m < 1 || a.m > MAXM || a.H < 1 || a.n_keys < 0)
        return CSD_ERR_INVALID_ARG;
    const int total = a.causal ? a.n_keys + a.m - 1 : a.n_keys;
    if (total < 1 || total > a.cap) return CSD_ERR_CAPACITY;
    AttnParams ap;
    ap.q = a.q; ap.Kc = a.Kc; ap.Vc = a.Vc; ap.bias = a.bias; ap.out = a.out; ap.partial = a.partial;
    ap.tickets = a.tickets; ap.ldq = a.ldq; ap.m = a.m; ap.cap = a.cap; ap.H = a.H; ap.n_keys = a.n_keys;
    ap.causal = a.causal; ap.bias_len = a.bias_len; ap.bias_zero = a.bias_zero; ap.q_pos0 = a.q_pos0;
    ap.ldo = a.ldo; ap.scale = a.scale; ap.out_xs = a.out_xs; ap.out_xs_ld = a.out_xs_ld;
    ap.nsplit = attn_splits(total, a.H);
    int len = (total + ap.nsplit - 1) / ap.nsplit;
    ap.split_len = (len + TILE - 1) / TILE * TILE;
    ap.nsplit = (total + ap.split_len - 1) / ap.split_len;
    if (ap.nsplit > 1 && (!a.partial || !a.tickets)) return CSD_ERR_INVALID_ARG;
    switch (a.Dh) {
        case 32: return launch_dh<32>(ap, st);
        case 64: return launch_dh<64>(ap, st);
        case 128: return launch_dh<128>(ap, st);
    }
    return CSD_ERR_SHAPE;
}

}  // namespace csd
