// Model handle and the review forward: one pass of a transformer over a block of m <= 17 rows
// that streams the bf16 weights once, reads the bf16 K/V cache and appends the block to it.
#include "model.cuh"
#include <math.h>
#include <new>
#include <stdlib.h>
#include <string.h>
#include <vector>

namespace csd {

// ---------------------------------------------------------------------------------------------
// small kernels
// ---------------------------------------------------------------------------------------------
__global__ void embed_kernel(const int32_t* __restrict__ tokens, const __nv_bfloat16* __restrict__ E, int V, int d,
                             float* __restrict__ x, int* status) {
    pdl_wait();
    pdl_trigger();
    const int r = blockIdx.x;
    int t = tokens[r];
    if (t < 0 || t >= V) {
        if (threadIdx.x == 0) set_status(status, CSD_ERR_BAD_TOKEN);
        t = 0;
    }
    const __nv_bfloat16* e = E + (size_t)t * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) x[(size_t)r * d + i] = __bfloat162float(e[i]);
}

// The same gather for a forward whose first projection runs on the tensor cores: besides the fp32 rows it
// writes the rows times `gain` as three bf16 terms (rows term * m + r of xs) and the pieces of each row's sum
// of squares, i.e. what the stand-alone split of those rows would write next.  grid = (d / 1024 rounded up, m).
__global__ void __launch_bounds__(128)
embed_split_kernel(const int32_t* __restrict__ tokens, const __nv_bfloat16* __restrict__ E, int V, int d, int m,
                   const __nv_bfloat16* __restrict__ gain, float* __restrict__ x, __nv_bfloat16* __restrict__ xs,
                   float* __restrict__ ssq, int* status) {
    pdl_wait();
    pdl_trigger();
    const int r = blockIdx.y, k = (blockIdx.x * 128 + threadIdx.x) * 8;
    int t = tokens[r];
    if (t < 0 || t >= V) {
        if (threadIdx.x == 0 && blockIdx.x == 0) set_status(status, CSD_ERR_BAD_TOKEN);
        t = 0;
    }
    float sq = 0.f;
    if (k < d) {
        const uint4 e = *reinterpret_cast<const uint4*>(E + (size_t)t * d + k);
        float v[8] = {bf16lo(e.x), bf16hi(e.x), bf16lo(e.y), bf16hi(e.y), bf16lo(e.z), bf16hi(e.z), bf16lo(e.w), bf16hi(e.w)};
        float* dst = x + (size_t)r * d + k;
        *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
        *reinterpret_cast<float4*>(dst + 4) = make_float4(v[4], v[5], v[6], v[7]);
#pragma unroll
        for (int i = 0; i < 8; ++i) sq = fmaf(v[i], v[i], sq);
        const uint4 g = *reinterpret_cast<const uint4*>(gain + k);
        v[0] *= bf16lo(g.x); v[1] *= bf16hi(g.x); v[2] *= bf16lo(g.y); v[3] *= bf16hi(g.y);
        v[4] *= bf16lo(g.z); v[5] *= bf16hi(g.z); v[6] *= bf16lo(g.w); v[7] *= bf16hi(g.w);
        uint32_t w[3][4];
#pragma unroll
        for (int i = 0; i < 8; i += 2) {
            uint16_t a1, a2, a3, c1, c2, c3;
            split3(v[i], a1, a2, a3);
            split3(v[i + 1], c1, c2, c3);
            w[0][i / 2] = a1 | ((uint32_t)c1 << 16); w[1][i / 2] = a2 | ((uint32_t)c2 << 16);
            w[2][i / 2] = a3 | ((uint32_t)c3 << 16);
        }
#pragma unroll
        for (int u = 0; u < 3; ++u)
            *reinterpret_cast<uint4*>(xs + (size_t)(u * m + r) * d + k) = make_uint4(w[u][0], w[u][1], w[u][2], w[u][3]);
    }
    __shared__ float part[4];
    sq = warp_sum(sq);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = sq;
    __syncthreads();
    if (threadIdx.x == 0) ssq[(size_t)blockIdx.x * m + r] = (part[0] + part[1]) + (part[2] + part[3]);
}

// cos/sin of pos * theta^(-2i/Dh), evaluated in double once per model
__global__ void rope_table_kernel(float* __restrict__ cs, float* __restrict__ sn, int max_seq, int half, double theta) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= max_seq * half) return;
    const int pos = idx / half, i = idx % half;
    const double ang = (double)pos * pow(theta, -(double)i / (double)half);
    cs[idx] = (float)cos(ang);
    sn[idx] = (float)sin(ang);
}

// bias_by_distance[h][i] = rel_bias[bucket[i]][h]
__global__ void bias_table_kernel(const __nv_bfloat16* __restrict__ rel_bias, const int* __restrict__ bucket, int len,
                                  int H, float* __restrict__ table) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= len * H) return;
    const int h = idx / len, i = idx % len;
    table[idx] = __bfloat162float(rel_bias[(size_t)bucket[i] * H + h]);
}

// Rotates q (in place) and k of the block's rows, then appends k and v to the cache as bf16.
// grid = (rows, heads); src is the fused projection output [rows, ld] with q|k|v column blocks.
__global__ void rope_append_kernel(float* __restrict__ src, int ld, int q_off, int k_off, int v_off, int Dh,
                                   int pos0, int cap, const float* __restrict__ cs, const float* __restrict__ sn,
                                   __nv_bfloat16* __restrict__ Kc, __nv_bfloat16* __restrict__ Vc) {
    pdl_wait();
    pdl_trigger();
    const int r = blockIdx.x, h = blockIdx.y, pos = pos0 + r, half = Dh / 2;
    float* row = src + (size_t)r * ld;
    __nv_bfloat16* kdst = Kc + ((size_t)h * cap + pos) * Dh;
    __nv_bfloat16* vdst = Vc + ((size_t)h * cap + pos) * Dh;
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
        float k0 = row[k_off + h * Dh + i], k1 = row[k_off + h * Dh + i + half];
        if (cs) {
            const float c = cs[(size_t)pos * half + i], s = sn[(size_t)pos * half + i];
            if (q_off >= 0) {
                float* q = row + q_off + h * Dh;
                const float q0 = q[i], q1 = q[i + half];
                q[i] = q0 * c - q1 * s;
                q[i + half] = q0 * s + q1 * c;
            }
            const float a = k0 * c - k1 * s, b = k0 * s + k1 * c;
            k0 = a; k1 = b;
        }
        kdst[i] = __float2bfloat16_rn(k0);
        kdst[i + half] = __float2bfloat16_rn(k1);
        vdst[i] = __float2bfloat16_rn(row[v_off + h * Dh + i]);
        vdst[i + half] = __float2bfloat16_rn(row[v_off + h * Dh + i + half]);
    }
}

// ---------------------------------------------------------------------------------------------
// layout helpers
// ---------------------------------------------------------------------------------------------
static size_t al128(size_t n) { return (n + 127) / 128 * 128; }

struct BlobWalk {
    const __nv_bfloat16* base;
    size_t off = 0;
    const __nv_bfloat16* take(size_t n) {
        const __nv_bfloat16* p = base ? base + off : nullptr;
        off = al128(off + n);
        return p;
    }
};

static void walk_attn(BlobWalk& w, size_t di, size_t d, const __nv_bfloat16*& q, const __nv_bfloat16*& k,
                      const __nv_bfloat16*& v, const __nv_bfloat16*& o) {
    q = w.take(di * d); k = w.take(di * d); v = w.take(di * d); o = w.take(d * di);
}

static size_t walk_blob(const csd_model_config& c, const __nv_bfloat16* base, csd_model* m) {
    BlobWalk w{base};
    const size_t d = c.d_model, di = (size_t)c.n_heads * c.d_head, ff = c.d_ff, V = c.vocab;
    const __nv_bfloat16* embed = w.take(V * d);
    std::vector<LayerW> enc, dec;
    const __nv_bfloat16 *enc_bias = nullptr, *dec_bias = nullptr, *enc_final = nullptr;
    if (c.arch == 1) {
        enc_bias = w.take((size_t)c.rel_buckets * c.n_heads);
        for (int l = 0; l < c.n_enc_layers; ++l) {
            LayerW y{};
            y.norm1 = w.take(d);
            walk_attn(w, di, d, y.wq, y.wk, y.wv, y.wo);
            y.norm2 = w.take(d); y.wgate = w.take(ff * d); y.wup = w.take(ff * d); y.wdown = w.take(d * ff);
            enc.push_back(y);
        }
        enc_final = w.take(d);
        dec_bias = w.take((size_t)c.rel_buckets * c.n_heads);
    }
    for (int l = 0; l < c.n_layers; ++l) {
        LayerW y{};
        y.norm1 = w.take(d);
        walk_attn(w, di, d, y.wq, y.wk, y.wv, y.wo);
        if (c.arch == 1) {
            y.norm_x = w.take(d);
            walk_attn(w, di, d, y.xq, y.xk, y.xv, y.xo);
        }
        y.norm2 = w.take(d); y.wgate = w.take(ff * d); y.wup = w.take(ff * d); y.wdown = w.take(d * ff);
        dec.push_back(y);
    }
    const __nv_bfloat16* final_norm = w.take(d);
    const __nv_bfloat16* lm_head = w.take(V * d);
    if (m) {
        m->embed = embed; m->enc = enc; m->dec = dec; m->enc_rel_bias = enc_bias; m->dec_rel_bias = dec_bias;
        m->enc_final_norm = enc_final; m->final_norm = final_norm; m->lm_head = lm_head;
    }
    return w.off;
}

struct WsLayout {
    size_t kcache, vcache, xk, xv, ek, ev, x, qkv, attn, act, xenc, qkv_enc, rope_c, rope_s, dec_bias, enc_bias,
        buckets, gemm_partial, gemm_tickets, xs_tmp, ssq_tmp, xs_x, xs_attn, xs_act, ssq_x,
        wx, wqkv, wattn, wact, wxs_x, wxs_attn, wxs_act, wssq, wpart, total;
    bool wide;
    size_t layer_kv, layer_x;
};

// The wide-block path serves a model when each of its layer matrices takes the wide kernel at 128 rows.
static bool wide_capable(const csd_model_config& c) {
    const int d = c.d_model, di = c.n_heads * c.d_head, ff = c.d_ff, R = CSD_WIDE_ROWS;
    return wide_supported(R, di, d, false) && wide_supported(R, 3 * di, d, false) && wide_supported(R, d, di, false) &&
           wide_supported(R, ff, d, true) && wide_supported(R, d, ff, false);
}

static WsLayout ws_layout(const csd_model_config& c) {
    WsLayout L{};
    const size_t d = c.d_model, H = c.n_heads, Dh = c.d_head, di = H * Dh, ff = c.d_ff, V = c.vocab;
    const size_t R = CSD_MAX_ROWS;
    size_t off = 0;
    auto put = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    L.layer_kv = H * (size_t)c.max_seq * Dh;
    L.kcache = put(c.n_layers * L.layer_kv * 2);
    L.vcache = put(c.n_layers * L.layer_kv * 2);
    L.x = put(R * d * 4);
    L.qkv = put(R * 3 * di * 4);
    L.attn = put(R * di * 4);
    L.act = put(R * ff * 4);
    size_t gp = 0, nmax = 0;
    auto mat = [&](size_t N, size_t K, bool dual) {
        size_t b = linear_scratch_bytes((int)R, (int)N, (int)K, dual);
        if (b > gp) gp = b;
        if (N > nmax) nmax = N;
    };
    mat(3 * di, d, false); mat(di, d, false); mat(d, di, false); mat(ff, d, true); mat(d, ff, false); mat(V, d, false);
    L.gemm_partial = put(gp);
    L.gemm_tickets = put((size_t)linear_ticket_count((int)nmax) * 4);
    const size_t kmax = d > di ? (d > ff ? d : ff) : (di > ff ? di : ff);
    L.xs_tmp = put(3 * R * kmax * 2);
    L.ssq_tmp = put((size_t)split_ssq_entries((int)kmax) * R * 4);
    L.xs_x = put(3 * R * d * 2);
    L.xs_attn = put(3 * R * di * 2);
    L.xs_act = put(3 * R * ff * 2);
    L.ssq_x = put((size_t)linear_ssq_capacity((int)d) * R * 4);
    L.wide = wide_capable(c);
    if (L.wide) {
        const size_t WR = CSD_WIDE_ROWS;
        L.wx = put(WR * d * 4); L.wqkv = put(WR * 3 * di * 4); L.wattn = put(WR * di * 4); L.wact = put(WR * ff * 4);
        L.wxs_x = put(2 * WR * d * 2); L.wxs_attn = put(2 * WR * di * 2); L.wxs_act = put(2 * WR * ff * 2);
        const size_t kmax_w = d > di ? (d > ff ? d : ff) : (di > ff ? di : ff);
        size_t pieces = (size_t)wide_ssq_capacity((int)d);
        if ((size_t)wide_split_pieces((int)kmax_w) > pieces) pieces = (size_t)wide_split_pieces((int)kmax_w);
        L.wssq = put(pieces * WR * 4);
        size_t pb = wide_partial_bytes((int)WR, (int)d, (int)di, false);
        if (wide_partial_bytes((int)WR, (int)d, (int)ff, false) > pb) pb = wide_partial_bytes((int)WR, (int)d, (int)ff, false);
        L.wpart = put(pb > 0 ? pb : 256);
    }
    if (c.arch == 0) {
        L.rope_c = put((size_t)c.max_seq * (Dh / 2) * 4);
        L.rope_s = put((size_t)c.max_seq * (Dh / 2) * 4);
    } else {
        const size_t E = c.max_enc_len;
        L.layer_x = H * E * Dh;
        L.xk = put(c.n_layers * L.layer_x * 2);
        L.xv = put(c.n_layers * L.layer_x * 2);
        L.ek = put(L.layer_x * 2);
        L.ev = put(L.layer_x * 2);
        L.xenc = put(E * d * 4);
        L.qkv_enc = put(E * 3 * di * 4);
        L.dec_bias = put(H * (size_t)c.max_seq * 4);
        L.enc_bias = put(H * (2 * E - 1) * 4);
        L.buckets = put((c.max_seq + 2 * E) * 4);
    }
    L.total = off;
    return L;
}

static csd_status check_config(const csd_model_config* c) {
    if (!c) return CSD_ERR_INVALID_ARG;
    if (c->arch != 0 && c->arch != 1) return CSD_ERR_UNSUPPORTED;
    if (c->n_layers < 1 || c->d_model < 8 || c->n_heads < 1 || c->d_ff < 8 || c->vocab < 1 || c->max_seq < 1)
        return CSD_ERR_INVALID_ARG;
    if (c->max_rows < 1 || c->max_rows > CSD_MAX_ROWS) return CSD_ERR_INVALID_ARG;
    if ((c->d_model & 7) || (c->d_ff & 7)) return CSD_ERR_SHAPE;
    if (c->d_head != 32 && c->d_head != 64 && c->d_head != 128) return CSD_ERR_SHAPE;
    if (c->arch == 1) {
        if (c->n_enc_layers < 1 || c->max_enc_len < 1 || c->rel_buckets < 4 || (c->rel_buckets & 3) ||
            c->rel_max_dist < c->rel_buckets)
            return CSD_ERR_INVALID_ARG;
    }
    return CSD_OK;
}

// Hand-over of activations between kernels on the tensor-core path: a GEMM may receive its rows
// already split into three bf16 terms (by the kernel that produced them) and may emit its own
// result in that form, times the gain of the norm that follows, with the pieces of the rows' sums
// of squares that norm needs.
struct LinOpt {
    const __nv_bfloat16* xs_in = nullptr; const float* ssq_in = nullptr; int ssq_cnt = 0;
    __nv_bfloat16* out_xs = nullptr; int out_ld = 0; const __nv_bfloat16* out_gain = nullptr; float* out_ssq = nullptr;
};

// One linear layer of the forward; all of them share the model's split scratch.
static csd_status linear(csd_model* M, const __nv_bfloat16* W, const __nv_bfloat16* W2, int N, int K, const float* X,
                         int ldx, int m, const __nv_bfloat16* gain, float* Y, int ldy, int epi, cudaStream_t st,
                         const LinOpt* o = nullptr) {
    LinearArgs a;
    a.W = W; a.W2 = W2; a.N = N; a.K = K; a.X = X; a.ldx = ldx; a.m = m; a.gain = gain; a.eps = M->cfg.norm_eps;
    a.Y = Y; a.ldy = ldy; a.epilogue = epi; a.partial = M->gemm_partial; a.tickets = M->gemm_tickets;
    a.xs = M->xs_tmp; a.ssq = M->ssq_tmp;
    if (o) {
        if (o->xs_in) {
            a.xs = const_cast<__nv_bfloat16*>(o->xs_in); a.xs_ready = true;
            a.ssq = const_cast<float*>(o->ssq_in); a.ssq_cnt = o->ssq_cnt;
        }
        a.out_xs = o->out_xs; a.out_ld = o->out_ld; a.out_gain = o->out_gain; a.out_ssq = o->out_ssq;
        if (o->out_ssq == M->ssq_x) M->ssq_x_cnt = linear_ssq_pieces(m, N, K, W2 != nullptr);
    }
    ProfScope ps(M, 0, st);
    if (M->prof) M->prof_gemm_bytes += (double)N * K * 2.0 * (W2 ? 2.0 : 1.0);
    return launch_linear(a, st);
}

#define CSD_TRY(expr)                       \
    do {                                    \
        csd_status s__ = (expr);            \
        if (s__ != CSD_OK) return s__;      \
    } while (0)

static csd_status attention(csd_model* M, const AttnArgs& a, cudaStream_t st) {
    ProfScope ps(M, 1, st);
    return launch_attention(a, st);
}

// q|k|v projections of `m` rows with the norm fused; one GEMM when the three matrices are
// contiguous in the blob (they are whenever d_inner * d_model is a multiple of 128).
static csd_status project_qkv(csd_model* M, const LayerW& y, const float* X, int m, float* out, cudaStream_t st,
                              const LinOpt* o = nullptr) {
    const int d = M->cfg.d_model, di = M->di;
    if (y.wk == y.wq + (size_t)di * d && y.wv == y.wk + (size_t)di * d)
        return linear(M, y.wq, nullptr, 3 * di, d, X, d, m, y.norm1, out, 3 * di, EPI_STORE, st, o);
    CSD_TRY(linear(M, y.wq, nullptr, di, d, X, d, m, y.norm1, out, 3 * di, EPI_STORE, st, o));
    CSD_TRY(linear(M, y.wk, nullptr, di, d, X, d, m, y.norm1, out + di, 3 * di, EPI_STORE, st, o));
    return linear(M, y.wv, nullptr, di, d, X, d, m, y.norm1, out + 2 * di, 3 * di, EPI_STORE, st, o);
}

// Gated feed-forward with its norm, then the down projection added into the residual rows.
// x_in: the rows already in three-term form (or null); next_gain: gain of the norm that reads the
// residual rows next (the result is handed on in three-term form when the kernels allow it).
// Returns through *x_out whether M->xs_x / M->ssq_x now describe the updated rows.
static csd_status feed_forward(csd_model* M, const LayerW& y, float* X, int m, cudaStream_t st,
                               bool x_in = false, const __nv_bfloat16* next_gain = nullptr, int next_N = 0,
                               bool next_dual = false, bool* x_out = nullptr) {
    const int d = M->cfg.d_model, ff = M->cfg.d_ff;
    const bool tc_up = linear_uses_tensor_cores(m, ff, d, true), tc_down = linear_uses_tensor_cores(m, d, ff, false);
    LinOpt up;
    if (x_in) { up.xs_in = M->xs_x; up.ssq_in = M->ssq_x; up.ssq_cnt = M->ssq_x_cnt; }
    const bool act_ready = tc_up && tc_down;
    if (act_ready) { up.out_xs = M->xs_act; up.out_ld = ff; }
    CSD_TRY(linear(M, y.wgate, y.wup, ff, d, X, d, m, y.norm2, M->act, ff, M->cfg.arch == 0 ? EPI_SWIGLU : EPI_GEGLU, st, &up));
    LinOpt down;
    if (act_ready) down.xs_in = M->xs_act;
    const bool hand_on = tc_down && next_gain && linear_uses_tensor_cores(m, next_N, d, next_dual);
    if (hand_on) { down.out_xs = M->xs_x; down.out_ld = d; down.out_gain = next_gain; down.out_ssq = M->ssq_x; }
    if (x_out) *x_out = hand_on;
    return linear(M, y.wdown, nullptr, d, ff, M->act, ff, m, nullptr, X, d, EPI_ADD, st, &down);
}

// ---------------------------------------------------------------------------------------------
// wide blocks: one pass of the decoder over up to CSD_WIDE_ROWS rows that only fills the cache
// ---------------------------------------------------------------------------------------------
static csd_status wide_linear(csd_model* M, const __nv_bfloat16* W, const __nv_bfloat16* W2, int N, int K, int m,
                              const __nv_bfloat16* xs, const float* ssq, int ssq_cnt, float* Y, int ldy, int epi,
                              __nv_bfloat16* out_xs, int out_ld, const __nv_bfloat16* out_gain, float* out_ssq,
                              cudaStream_t st) {
    WideArgs a;
    a.W = W; a.W2 = W2; a.N = N; a.K = K; a.m = m; a.xs = xs; a.ssq = ssq; a.ssq_cnt = ssq_cnt; a.eps = M->cfg.norm_eps;
    a.Y = Y; a.ldy = ldy; a.epilogue = epi; a.out_xs = out_xs; a.out_ld = out_ld; a.out_gain = out_gain; a.out_ssq = out_ssq;
    a.partial = M->wpart;
    ProfScope ps(M, 0, st);
    if (M->prof) M->prof_gemm_bytes += (double)N * K * 2.0 * (W2 ? 2.0 : 1.0);
    return launch_linear_wide(a, st);
}

// Attention of `m` <= CSD_WIDE_ROWS rows over K/V that are already in the cache: row r sees keys
// [0, n_keys0 + r) when causal, all n_keys0 otherwise.
static csd_status wide_attention(csd_model* M, const float* q, int ldq, int m, __nv_bfloat16* Kc, __nv_bfloat16* Vc, int cap,
                                 int n_keys0, bool causal, const float* bias, int bias_len, int bias_zero, int q_pos0,
                                 float* out, cudaStream_t st) {
    const csd_model_config& c = M->cfg;
    AttnArgs a;       // one launch over all rows where the tensor-core kernel applies (sub-blocks in its grid)
    a.q = q; a.ldq = ldq; a.m = m;
    a.Kc = Kc; a.Vc = Vc; a.cap = cap; a.H = c.n_heads; a.Dh = c.d_head;
    a.n_keys = n_keys0; a.causal = causal ? 1 : 0;
    a.scale = c.arch == 0 ? 1.f / sqrtf((float)c.d_head) : 1.f;
    a.bias = bias; a.bias_len = bias_len; a.bias_zero = bias_zero; a.q_pos0 = q_pos0;
    a.out = out; a.ldo = M->di;
    return attention(M, a, st);
}

// Decoder pass over m <= CSD_WIDE_ROWS rows at positions kv_len .. kv_len+m-1: K/V of every layer are
// appended, nothing else is kept.
static csd_status wide_decoder_pass(csd_model* M, const int32_t* tokens, int m, int kv_len, cudaStream_t st) {
    const csd_model_config& c = M->cfg;
    const int d = c.d_model, H = c.n_heads, Dh = c.d_head, di = M->di, ff = c.d_ff;
    {
        ProfScope ps(M, 2, st);
        embed_kernel<<<m, 128, 0, st>>>(tokens, M->embed, c.vocab, d, M->wx, M->status);
        count_launch();
    }
    int cnt = 0;                       // pieces in wssq that describe the rows in wxs_x (0: wxs_x not current)
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerW& y = M->dec[l];
        __nv_bfloat16* Kl = M->kcache + (size_t)l * M->layer_kv;
        __nv_bfloat16* Vl = M->vcache + (size_t)l * M->layer_kv;
        if (cnt == 0) {
            CSD_TRY(launch_wide_split(M->wx, d, d, m, y.norm1, M->wxs_x, M->wssq, st));
            cnt = wide_split_pieces(d);
        }
        if (y.wk == y.wq + (size_t)di * d && y.wv == y.wk + (size_t)di * d) {
            CSD_TRY(wide_linear(M, y.wq, nullptr, 3 * di, d, m, M->wxs_x, M->wssq, cnt, M->wqkv, 3 * di, EPI_STORE, nullptr, 0,
                                nullptr, nullptr, st));
        } else {
            const __nv_bfloat16* w3[3] = {y.wq, y.wk, y.wv};
            for (int i = 0; i < 3; ++i)
                CSD_TRY(wide_linear(M, w3[i], nullptr, di, d, m, M->wxs_x, M->wssq, cnt, M->wqkv + (size_t)i * di, 3 * di,
                                    EPI_STORE, nullptr, 0, nullptr, nullptr, st));
        }
        {   // rotate q and k, append k and v of all rows; the sub-blocks below then only read the cache
            ProfScope ps(M, 2, st);
            rope_append_kernel<<<dim3(m, H), 64, 0, st>>>(M->wqkv, 3 * di, c.arch == 0 ? 0 : -1, di, 2 * di, Dh, kv_len, c.max_seq,
                                                          c.arch == 0 ? M->rope_c : nullptr, c.arch == 0 ? M->rope_s : nullptr, Kl, Vl);
            count_launch();
        }
        if (l + 1 == c.n_layers) break;    // the cache is complete; the rest of the last layer feeds nothing
        CSD_TRY(wide_attention(M, M->wqkv, 3 * di, m, Kl, Vl, c.max_seq, kv_len + 1, true,
                               c.arch == 1 ? M->dec_bias : nullptr, c.max_seq, c.max_seq - 1, kv_len, M->wattn, st));
        CSD_TRY(launch_wide_split(M->wattn, di, di, m, nullptr, M->wxs_attn, nullptr, st));
        const __nv_bfloat16* after_o = c.arch == 1 ? y.norm_x : y.norm2;
        CSD_TRY(wide_linear(M, y.wo, nullptr, d, di, m, M->wxs_attn, nullptr, 0, M->wx, d, EPI_ADD, M->wxs_x, d, after_o,
                            M->wssq, st));
        cnt = wide_ssq_pieces(m, d, di, false);
        if (c.arch == 1) {
            CSD_TRY(wide_linear(M, y.xq, nullptr, di, d, m, M->wxs_x, M->wssq, cnt, M->wqkv, 3 * di, EPI_STORE, nullptr, 0,
                                nullptr, nullptr, st));
            CSD_TRY(wide_attention(M, M->wqkv, 3 * di, m, M->xk + (size_t)l * M->layer_x, M->xv + (size_t)l * M->layer_x,
                                   c.max_enc_len, M->enc_len, false, nullptr, 0, 0, 0, M->wattn, st));
            CSD_TRY(launch_wide_split(M->wattn, di, di, m, nullptr, M->wxs_attn, nullptr, st));
            CSD_TRY(wide_linear(M, y.xo, nullptr, d, di, m, M->wxs_attn, nullptr, 0, M->wx, d, EPI_ADD, M->wxs_x, d, y.norm2,
                                M->wssq, st));
            cnt = wide_ssq_pieces(m, d, di, false);
        }
        CSD_TRY(wide_linear(M, y.wgate, y.wup, ff, d, m, M->wxs_x, M->wssq, cnt, M->wact, ff,
                            c.arch == 0 ? EPI_SWIGLU : EPI_GEGLU, M->wxs_act, ff, nullptr, nullptr, st));
        CSD_TRY(wide_linear(M, y.wdown, nullptr, d, ff, m, M->wxs_act, nullptr, 0, M->wx, d, EPI_ADD, M->wxs_x, d,
                            M->dec[l + 1].norm1, M->wssq, st));
        cnt = wide_ssq_pieces(m, d, ff, false);
    }
    CSD_CUDA(cudaGetLastError());
    return CSD_OK;
}

// Encoder pass (arch 1) in wide blocks: every layer projects q|k|v of all rows, appends K/V, then
// runs attention, output projection and feed-forward block by block; afterwards the cross-attention
// K/V of every decoder layer.
static csd_status wide_encoder(csd_model* M, int n, cudaStream_t st) {
    const csd_model_config& c = M->cfg;
    const int d = c.d_model, H = c.n_heads, Dh = c.d_head, di = M->di, ff = c.d_ff, E = c.max_enc_len, WR = CSD_WIDE_ROWS;
    for (int l = 0; l < c.n_enc_layers; ++l) {
        const LayerW& y = M->enc[l];
        const bool fused = y.wk == y.wq + (size_t)di * d && y.wv == y.wk + (size_t)di * d;
        for (int r0 = 0; r0 < n; r0 += WR) {
            const int m = n - r0 < WR ? n - r0 : WR;
            CSD_TRY(launch_wide_split(M->xenc + (size_t)r0 * d, d, d, m, y.norm1, M->wxs_x, M->wssq, st));
            const int cnt = wide_split_pieces(d);
            float* out = M->qkv_enc + (size_t)r0 * 3 * di;
            if (fused) {
                CSD_TRY(wide_linear(M, y.wq, nullptr, 3 * di, d, m, M->wxs_x, M->wssq, cnt, out, 3 * di, EPI_STORE, nullptr, 0,
                                    nullptr, nullptr, st));
            } else {
                const __nv_bfloat16* w3[3] = {y.wq, y.wk, y.wv};
                for (int i = 0; i < 3; ++i)
                    CSD_TRY(wide_linear(M, w3[i], nullptr, di, d, m, M->wxs_x, M->wssq, cnt, out + (size_t)i * di, 3 * di,
                                        EPI_STORE, nullptr, 0, nullptr, nullptr, st));
            }
        }
        rope_append_kernel<<<dim3(n, H), 64, 0, st>>>(M->qkv_enc, 3 * di, -1, di, 2 * di, Dh, 0, E, nullptr, nullptr, M->ek, M->ev);
        count_launch();
        for (int r0 = 0; r0 < n; r0 += WR) {
            const int m = n - r0 < WR ? n - r0 : WR;
            float* xr = M->xenc + (size_t)r0 * d;
            CSD_TRY(wide_attention(M, M->qkv_enc + (size_t)r0 * 3 * di, 3 * di, m, M->ek, M->ev, E, n, false, M->enc_bias,
                                   2 * E - 1, E - 1, r0, M->wattn, st));
            CSD_TRY(launch_wide_split(M->wattn, di, di, m, nullptr, M->wxs_attn, nullptr, st));
            CSD_TRY(wide_linear(M, y.wo, nullptr, d, di, m, M->wxs_attn, nullptr, 0, xr, d, EPI_ADD, M->wxs_x, d, y.norm2,
                                M->wssq, st));
            CSD_TRY(wide_linear(M, y.wgate, y.wup, ff, d, m, M->wxs_x, M->wssq, wide_ssq_pieces(m, d, di, false), M->wact, ff,
                                EPI_GEGLU, M->wxs_act, ff, nullptr, nullptr, st));
            CSD_TRY(wide_linear(M, y.wdown, nullptr, d, ff, m, M->wxs_act, nullptr, 0, xr, d, EPI_ADD, nullptr, 0, nullptr,
                                nullptr, st));
        }
    }
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerW& y = M->dec[l];
        for (int r0 = 0; r0 < n; r0 += WR) {
            const int m = n - r0 < WR ? n - r0 : WR;
            CSD_TRY(launch_wide_split(M->xenc + (size_t)r0 * d, d, d, m, M->enc_final_norm, M->wxs_x, M->wssq, st));
            const int cnt = wide_split_pieces(d);
            float* out = M->qkv_enc + (size_t)r0 * 3 * di;
            CSD_TRY(wide_linear(M, y.xk, nullptr, di, d, m, M->wxs_x, M->wssq, cnt, out + di, 3 * di, EPI_STORE, nullptr, 0, nullptr,
                                nullptr, st));
            CSD_TRY(wide_linear(M, y.xv, nullptr, di, d, m, M->wxs_x, M->wssq, cnt, out + 2 * di, 3 * di, EPI_STORE, nullptr, 0,
                                nullptr, nullptr, st));
        }
        rope_append_kernel<<<dim3(n, H), 64, 0, st>>>(M->qkv_enc, 3 * di, -1, di, 2 * di, Dh, 0, E, nullptr, nullptr,
                                                      M->xk + (size_t)l * M->layer_x, M->xv + (size_t)l * M->layer_x);
        count_launch();
    }
    CSD_CUDA(cudaGetLastError());
    return CSD_OK;
}

}  // namespace csd

using namespace csd;

extern "C" int csd_rel_bucket(int rel, int bidirectional, int n_buckets, int max_dist) {
    int bucket = 0, B = n_buckets, n;
    if (bidirectional) {
        B /= 2;
        if (rel > 0) bucket += B;
        n = rel < 0 ? -rel : rel;
    } else {
        n = rel < 0 ? -rel : 0;
    }
    const int exact = B / 2;
    if (n < exact) return bucket + n;
    // logarithmic part; the tiny nudge keeps distances that sit exactly on a bucket edge
    // (powers of two) on the upper side, as exact arithmetic puts them
    double t = log((double)n / exact) / log((double)max_dist / exact) * (B - exact);
    int b = exact + (int)floor(t + 1e-9);
    if (b > B - 1) b = B - 1;
    return bucket + b;
}

extern "C" size_t csd_model_weight_bytes(const csd_model_config* cfg) {
    if (check_config(cfg) != CSD_OK) return 0;
    return walk_blob(*cfg, nullptr, nullptr) * sizeof(__nv_bfloat16);
}

extern "C" size_t csd_model_workspace_bytes(const csd_model_config* cfg) {
    if (check_config(cfg) != CSD_OK) return 0;
    return ws_layout(*cfg).total;
}

extern "C" csd_status csd_model_create(const csd_model_config* cfg, const void* weights_bf16_dev, size_t weight_bytes,
                                       void* workspace_dev, size_t workspace_bytes, void* stream, csd_model** out) {
    if (!out) return CSD_ERR_INVALID_ARG;
    *out = nullptr;
    CSD_TRY(check_config(cfg));
    if (!weights_bf16_dev || !workspace_dev) return CSD_ERR_INVALID_ARG;
    if ((((uintptr_t)weights_bf16_dev) & 255) || (((uintptr_t)workspace_dev) & 255)) return CSD_ERR_INVALID_ARG;
    if (weight_bytes < csd_model_weight_bytes(cfg)) return CSD_ERR_CAPACITY;
    const WsLayout L = ws_layout(*cfg);
    if (workspace_bytes < L.total) return CSD_ERR_CAPACITY;
    int* status = status_word_device();
    if (!status) return CSD_ERR_CUDA;
    csd_model* M = new (std::nothrow) csd_model();
    if (!M) return CSD_ERR_OOM;
    M->cfg = *cfg;
    M->di = cfg->n_heads * cfg->d_head;
    walk_blob(*cfg, (const __nv_bfloat16*)weights_bf16_dev, M);
    char* ws = (char*)workspace_dev;
    M->kcache = (__nv_bfloat16*)(ws + L.kcache); M->vcache = (__nv_bfloat16*)(ws + L.vcache);
    M->layer_kv = L.layer_kv; M->layer_x = L.layer_x;
    M->x = (float*)(ws + L.x); M->qkv = (float*)(ws + L.qkv); M->attn = (float*)(ws + L.attn);
    M->act = (float*)(ws + L.act);
    M->gemm_partial = (float*)(ws + L.gemm_partial); M->gemm_tickets = (unsigned*)(ws + L.gemm_tickets);
    M->xs_tmp = (__nv_bfloat16*)(ws + L.xs_tmp); M->ssq_tmp = (float*)(ws + L.ssq_tmp);
    M->xs_x = (__nv_bfloat16*)(ws + L.xs_x); M->xs_attn = (__nv_bfloat16*)(ws + L.xs_attn);
    M->xs_act = (__nv_bfloat16*)(ws + L.xs_act); M->ssq_x = (float*)(ws + L.ssq_x);
    M->status = status;
    M->wide = L.wide;
    if (L.wide) {
        M->wx = (float*)(ws + L.wx); M->wqkv = (float*)(ws + L.wqkv); M->wattn = (float*)(ws + L.wattn);
        M->wact = (float*)(ws + L.wact); M->wxs_x = (__nv_bfloat16*)(ws + L.wxs_x);
        M->wxs_attn = (__nv_bfloat16*)(ws + L.wxs_attn); M->wxs_act = (__nv_bfloat16*)(ws + L.wxs_act);
        M->wssq = (float*)(ws + L.wssq); M->wpart = (float*)(ws + L.wpart);
    }
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = cudaMemsetAsync(ws + L.gemm_tickets, 0, L.xs_tmp - L.gemm_tickets, st);
    if (e != cudaSuccess) { delete M; return note_cuda(e); }
    if (cfg->arch == 0) {
        M->rope_c = (float*)(ws + L.rope_c); M->rope_s = (float*)(ws + L.rope_s);
        const int n = cfg->max_seq * (cfg->d_head / 2);
        rope_table_kernel<<<(n + 255) / 256, 256, 0, st>>>(M->rope_c, M->rope_s, cfg->max_seq, cfg->d_head / 2,
                                                           (double)cfg->rope_theta);
        count_launch();
    } else {
        const int E = cfg->max_enc_len, S = cfg->max_seq;
        M->xk = (__nv_bfloat16*)(ws + L.xk); M->xv = (__nv_bfloat16*)(ws + L.xv);
        M->ek = (__nv_bfloat16*)(ws + L.ek); M->ev = (__nv_bfloat16*)(ws + L.ev);
        M->xenc = (float*)(ws + L.xenc); M->qkv_enc = (float*)(ws + L.qkv_enc);
        M->dec_bias = (float*)(ws + L.dec_bias); M->enc_bias = (float*)(ws + L.enc_bias);
        int* buckets = (int*)(ws + L.buckets);
        std::vector<int> hb((size_t)S + 2 * E - 1);
        // decoder: index i <-> rel = i - (S-1) in [-(S-1), 0]; encoder: rel = i - (E-1) in [-(E-1), E-1]
        for (int i = 0; i < S; ++i) hb[i] = csd_rel_bucket(i - (S - 1), 0, cfg->rel_buckets, cfg->rel_max_dist);
        for (int i = 0; i < 2 * E - 1; ++i)
            hb[S + i] = csd_rel_bucket(i - (E - 1), 1, cfg->rel_buckets, cfg->rel_max_dist);
        e = cudaMemcpyAsync(buckets, hb.data(), hb.size() * sizeof(int), cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);   // hb goes out of scope below
        if (e != cudaSuccess) { delete M; return note_cuda(e); }
        bias_table_kernel<<<(S * cfg->n_heads + 255) / 256, 256, 0, st>>>(M->dec_rel_bias, buckets, S, cfg->n_heads, M->dec_bias);
        bias_table_kernel<<<((2 * E - 1) * cfg->n_heads + 255) / 256, 256, 0, st>>>(M->enc_rel_bias, buckets + S, 2 * E - 1,
                                                                                 cfg->n_heads, M->enc_bias);
        count_launch(2);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) { delete M; return note_cuda(e); }
    *out = M;
    return CSD_OK;
}

extern "C" csd_status csd_model_destroy(csd_model* m) {
    if (m)
        for (cudaEvent_t e : m->prof_ev) cudaEventDestroy(e);
    delete m;
    return CSD_OK;
}

extern "C" csd_status csd_model_profile(csd_model* m, int enable) {
    if (!m) return CSD_ERR_INVALID_ARG;
    m->prof = enable != 0;
    m->prof_used = 0;
    m->prof_gemm_bytes = 0.0;
    return CSD_OK;
}

extern "C" csd_status csd_model_profile_read(csd_model* m, void* stream, csd_profile* out) {
    if (!m || !out) return CSD_ERR_INVALID_ARG;
    CSD_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    csd_profile p;
    memset(&p, 0, sizeof(p));
    for (size_t i = 0; i < m->prof_used; ++i) {
        float ms = 0.f;
        CSD_CUDA(cudaEventElapsedTime(&ms, m->prof_ev[2 * i], m->prof_ev[2 * i + 1]));
        const int k = m->prof_kind[i];
        if (k == 0) { p.gemm_ms += ms; p.gemm_launches += 1; }
        else if (k == 1) { p.attn_ms += ms; p.attn_launches += 1; }
        else { p.other_ms += ms; p.other_launches += 1; }
    }
    p.gemm_weight_bytes = m->prof_gemm_bytes;
    m->prof_used = 0;
    m->prof_gemm_bytes = 0.0;
    *out = p;
    return CSD_OK;
}

extern "C" csd_status csd_encoder_forward(csd_model* M, const int32_t* enc_tokens_dev, int n, void* stream) {
    if (!M || !enc_tokens_dev) return CSD_ERR_INVALID_ARG;
    const csd_model_config& c = M->cfg;
    if (c.arch != 1) return CSD_ERR_UNSUPPORTED;
    if (n < 1 || n > c.max_enc_len) return CSD_ERR_CAPACITY;
    cudaStream_t st = (cudaStream_t)stream;
    const int d = c.d_model, H = c.n_heads, Dh = c.d_head, di = M->di, E = c.max_enc_len;
    const int CH = 16;
    embed_kernel<<<n, 128, 0, st>>>(enc_tokens_dev, M->embed, c.vocab, d, M->xenc, M->status);
    count_launch();
    if (M->wide && gemm_path() != 1 && n > CSD_MAX_ROWS) {      // large model: wide blocks
        CSD_TRY(wide_encoder(M, n, st));
        M->enc_len = n;
        return CSD_OK;
    }
    for (int l = 0; l < c.n_enc_layers; ++l) {
        const LayerW& y = M->enc[l];
        for (int r0 = 0; r0 < n; r0 += CH) {
            const int m = n - r0 < CH ? n - r0 : CH;
            CSD_TRY(project_qkv(M, y, M->xenc + (size_t)r0 * d, m, M->qkv_enc + (size_t)r0 * 3 * di, st));
        }
        rope_append_kernel<<<dim3(n, H), 64, 0, st>>>(M->qkv_enc, 3 * di, -1, di, 2 * di, Dh, 0, E, nullptr, nullptr,
                                                      M->ek, M->ev);
        count_launch();
        for (int r0 = 0; r0 < n; r0 += CH) {
            const int m = n - r0 < CH ? n - r0 : CH;
            AttnArgs a;
            a.q = M->qkv_enc + (size_t)r0 * 3 * di; a.ldq = 3 * di; a.m = m; a.Kc = M->ek; a.Vc = M->ev; a.cap = E;
            a.H = H; a.Dh = Dh; a.n_keys = n; a.causal = 0; a.scale = 1.f; a.bias = M->enc_bias;
            a.bias_len = 2 * E - 1; a.bias_zero = E - 1; a.q_pos0 = r0; a.out = M->attn; a.ldo = di;
            CSD_TRY(attention(M, a, st));
            float* xr = M->xenc + (size_t)r0 * d;
            CSD_TRY(linear(M, y.wo, nullptr, d, di, M->attn, di, m, nullptr, xr, d, EPI_ADD, st));
            CSD_TRY(feed_forward(M, y, xr, m, st));
        }
    }
    // static cross-attention K/V of every decoder layer from the normed encoder output
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerW& y = M->dec[l];
        for (int r0 = 0; r0 < n; r0 += CH) {
            const int m = n - r0 < CH ? n - r0 : CH;
            const float* xr = M->xenc + (size_t)r0 * d;
            float* o = M->qkv_enc + (size_t)r0 * 3 * di;
            CSD_TRY(linear(M, y.xk, nullptr, di, d, xr, d, m, M->enc_final_norm, o + di, 3 * di, EPI_STORE, st));
            CSD_TRY(linear(M, y.xv, nullptr, di, d, xr, d, m, M->enc_final_norm, o + 2 * di, 3 * di, EPI_STORE, st));
        }
        rope_append_kernel<<<dim3(n, H), 64, 0, st>>>(M->qkv_enc, 3 * di, -1, di, 2 * di, Dh, 0, E, nullptr, nullptr,
                                                      M->xk + (size_t)l * M->layer_x, M->xv + (size_t)l * M->layer_x);
        count_launch();
    }
    CSD_CUDA(cudaGetLastError());
    M->enc_len = n;
    return CSD_OK;
}

extern "C" csd_status csd_prefill(csd_model* M, const int32_t* tokens_dev, int n, int kv_len, void* stream) {
    if (!M || !tokens_dev || n < 1 || kv_len < 0) return CSD_ERR_INVALID_ARG;
    const csd_model_config& c = M->cfg;
    if (kv_len + n > c.max_seq) return CSD_ERR_CAPACITY;
    if (c.arch == 1 && M->enc_len < 1) return CSD_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const int small = c.max_rows < CSD_MAX_ROWS ? c.max_rows : CSD_MAX_ROWS;
    for (int from = 0; from < n;) {
        int cnt = n - from;
        // wide passes while more than one review block is left, review-sized blocks otherwise
        if (M->wide && gemm_path() != 1 && cnt > small) {
            if (cnt > CSD_WIDE_ROWS) cnt = CSD_WIDE_ROWS;
            CSD_TRY(wide_decoder_pass(M, tokens_dev + from, cnt, kv_len + from, st));
        } else {
            if (cnt > small) cnt = small;
            CSD_TRY(csd_review_forward(M, tokens_dev + from, cnt, kv_len + from, nullptr, stream));
        }
        from += cnt;
    }
    return CSD_OK;
}

// A block may hold the rows of several sequences (batched review): the contractions run once over
// all rows, the attention per sequence over that sequence's own cache.
struct Segment { csd_model* S; int row0, rows, kv_len; };
static csd_status review_forward_impl(csd_model* M, const int32_t* block_tokens_dev, int m, int kv_len,
                                      float* logits_out_dev, void* stream, const unsigned* tree_mask, const int* tree_depth,
                                      const Segment* segs = nullptr, int nseg = 0);

extern "C" csd_status csd_review_forward(csd_model* M, const int32_t* block_tokens_dev, int m, int kv_len,
                                         float* logits_out_dev, void* stream) {
    return review_forward_impl(M, block_tokens_dev, m, kv_len, logits_out_dev, stream, nullptr, nullptr);
}

extern "C" csd_status csd_review_forward_batch(csd_model* const* models, int n_seqs, const int32_t* block_tokens_dev,
                                               const int32_t* n_rows_host, const int32_t* kv_len_host,
                                               float* logits_out_dev, void* stream) {
    if (!models || n_seqs < 1 || n_seqs > CSD_MAX_ROWS || !block_tokens_dev || !n_rows_host || !kv_len_host)
        return CSD_ERR_INVALID_ARG;
    csd_model* M = models[0];
    if (!M) return CSD_ERR_INVALID_ARG;
    Segment segs[CSD_MAX_ROWS];
    int total = 0;
    for (int g = 0; g < n_seqs; ++g) {
        csd_model* S = models[g];
        // one set of weights, one shape: the handles differ in their caches only
        if (!S || S->embed != M->embed || memcmp(&S->cfg, &M->cfg, sizeof(M->cfg)) != 0) return CSD_ERR_INVALID_ARG;
        for (int h = 0; h < g; ++h)
            if (models[h] == S) return CSD_ERR_INVALID_ARG;
        const int rows = n_rows_host[g], kv = kv_len_host[g];
        if (rows < 1 || kv < 0) return CSD_ERR_INVALID_ARG;
        if (kv + rows > M->cfg.max_seq) return CSD_ERR_CAPACITY;
        if (M->cfg.arch == 1 && S->enc_len < 1) return CSD_ERR_INVALID_ARG;
        segs[g] = Segment{S, total, rows, kv};
        total += rows;
    }
    if (total > M->cfg.max_rows) return CSD_ERR_INVALID_ARG;
    return review_forward_impl(M, block_tokens_dev, total, segs[0].kv_len, logits_out_dev, stream, nullptr, nullptr, segs, n_seqs);
}

extern "C" csd_status csd_review_forward_tree(csd_model* M, const int32_t* block_tokens_dev, const int32_t* parent_host,
                                              int m, int kv_len, float* logits_out_dev, void* stream) {
    if (!M || !parent_host || m < 1 || m > CSD_MAX_ROWS) return CSD_ERR_INVALID_ARG;
    if (M->cfg.arch != 0) return CSD_ERR_UNSUPPORTED;         // positions enter through the rotary embedding only
    unsigned mask[CSD_MAX_ROWS];
    int depth[CSD_MAX_ROWS];
    for (int r = 0; r < m; ++r) {
        const int p = parent_host[r];
        if (r == 0 ? p != -1 : (p < 0 || p >= r)) return CSD_ERR_INVALID_ARG;   // row 0 is the root, parents come first
        mask[r] = (r == 0 ? 0u : mask[p]) | (1u << r);
        depth[r] = r == 0 ? 0 : depth[p] + 1;
    }
    if (kv_len + m > M->cfg.max_seq) return CSD_ERR_CAPACITY;
    return review_forward_impl(M, block_tokens_dev, m, kv_len, logits_out_dev, stream, mask, depth);
}

static csd_status review_forward_impl(csd_model* M, const int32_t* block_tokens_dev, int m, int kv_len,
                                      float* logits_out_dev, void* stream, const unsigned* tree_mask, const int* tree_depth,
                                      const Segment* segs, int nseg) {
    if (!M || !block_tokens_dev) return CSD_ERR_INVALID_ARG;
    const Segment whole{M, 0, m, kv_len};
    if (!segs) { segs = &whole; nseg = 1; }
    const csd_model_config& c = M->cfg;
    if (m < 1 || m > c.max_rows || kv_len < 0) return CSD_ERR_INVALID_ARG;
    if (kv_len + m > c.max_seq) return CSD_ERR_CAPACITY;
    if (c.arch == 1 && M->enc_len < 1) return CSD_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const int d = c.d_model, H = c.n_heads, Dh = c.d_head, di = M->di, V = c.vocab;
    // x_ready: M->xs_x / M->ssq_x hold the residual rows (times the gain of the norm that reads them
    // next) in three-term form, written by the epilogue of the GEMM that produced the rows (for the
    // embedded rows: by the gather itself, when the first projection takes that form)
    bool x_ready = false;
    {
        ProfScope ps(M, 2, st);
        const LayerW& y0 = M->dec[0];
        const bool fused_qkv = y0.wk == y0.wq + (size_t)di * d && y0.wv == y0.wk + (size_t)di * d;
        if ((d & 7) == 0 && linear_uses_tensor_cores(m, fused_qkv ? 3 * di : di, d, false)) {
            embed_split_kernel<<<dim3((unsigned)split_ssq_entries(d), (unsigned)m), 128, 0, st>>>(
                block_tokens_dev, M->embed, V, d, m, y0.norm1, M->x, M->xs_x, M->ssq_x, M->status);
            M->ssq_x_cnt = split_ssq_entries(d);
            x_ready = true;
        } else {
            embed_kernel<<<m, 128, 0, st>>>(block_tokens_dev, M->embed, V, d, M->x, M->status);
        }
        count_launch();
    }
    const int ff = c.d_ff;
    const bool tc_o = linear_uses_tensor_cores(m, d, di, false);
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerW& y = M->dec[l];
        __nv_bfloat16* Kl = M->kcache + (size_t)l * M->layer_kv;
        __nv_bfloat16* Vl = M->vcache + (size_t)l * M->layer_kv;
        {
            LinOpt qo;
            if (x_ready) { qo.xs_in = M->xs_x; qo.ssq_in = M->ssq_x; qo.ssq_cnt = M->ssq_x_cnt; }
            CSD_TRY(project_qkv(M, y, M->x, m, M->qkv, st, &qo));
        }
        for (int g = 0; g < nseg; ++g) {
            const Segment& sg = segs[g];
            AttnArgs a;
            a.q = M->qkv + (size_t)sg.row0 * 3 * di; a.ldq = 3 * di; a.m = sg.rows;
            a.Kc = sg.S->kcache + (size_t)l * sg.S->layer_kv; a.Vc = sg.S->vcache + (size_t)l * sg.S->layer_kv;
            a.cap = c.max_seq; a.H = H; a.Dh = Dh;
            a.n_keys = sg.kv_len + 1; a.causal = 1; a.scale = c.arch == 0 ? 1.f / sqrtf((float)Dh) : 1.f;
            if (c.arch == 1) { a.bias = M->dec_bias; a.bias_len = c.max_seq; a.bias_zero = c.max_seq - 1; a.q_pos0 = sg.kv_len; }
            a.out = M->attn + (size_t)sg.row0 * di; a.ldo = di;
            // the block's own k and v rows go into the cache inside the attention kernel
            a.k_new = a.q + di; a.v_new = a.q + 2 * di; a.ld_new = 3 * di;
            a.kv_settled = true;      // committed rows date from earlier forwards
            if (c.arch == 0) { a.rope_cos = M->rope_c; a.rope_sin = M->rope_s; }
            a.tree_mask = tree_mask; a.tree_depth = tree_depth;
            if (tc_o) { a.out_xs = M->xs_attn; a.out_xs_ld = di; a.out_xs_rows = m; a.out_xs_row0 = sg.row0; }
            CSD_TRY(attention(M, a, st));
        }
        // output projection into the residual rows; hands them on to the norm that follows
        LinOpt oo;
        if (tc_o) oo.xs_in = M->xs_attn;
        const __nv_bfloat16* after_o = c.arch == 1 ? y.norm_x : y.norm2;
        x_ready = tc_o && (c.arch == 1 ? linear_uses_tensor_cores(m, di, d, false) : linear_uses_tensor_cores(m, ff, d, true));
        if (x_ready) { oo.out_xs = M->xs_x; oo.out_ld = d; oo.out_gain = after_o; oo.out_ssq = M->ssq_x; }
        CSD_TRY(linear(M, y.wo, nullptr, d, di, M->attn, di, m, nullptr, M->x, d, EPI_ADD, st, &oo));
        if (c.arch == 1) {
            LinOpt xq;
            if (x_ready) { xq.xs_in = M->xs_x; xq.ssq_in = M->ssq_x; xq.ssq_cnt = M->ssq_x_cnt; }
            CSD_TRY(linear(M, y.xq, nullptr, di, d, M->x, d, m, y.norm_x, M->qkv, 3 * di, EPI_STORE, st, &xq));
            for (int g = 0; g < nseg; ++g) {
                const Segment& sg = segs[g];
                AttnArgs x;
                x.q = M->qkv + (size_t)sg.row0 * 3 * di; x.ldq = 3 * di; x.m = sg.rows;
                x.Kc = sg.S->xk + (size_t)l * sg.S->layer_x; x.Vc = sg.S->xv + (size_t)l * sg.S->layer_x;
                x.cap = c.max_enc_len; x.H = H; x.Dh = Dh; x.n_keys = sg.S->enc_len;
                x.causal = 0; x.scale = 1.f; x.out = M->attn + (size_t)sg.row0 * di; x.ldo = di;
                x.kv_settled = true;  // written once by the encoder pass
                if (tc_o) { x.out_xs = M->xs_attn; x.out_xs_ld = di; x.out_xs_rows = m; x.out_xs_row0 = sg.row0; }
                CSD_TRY(attention(M, x, st));
            }
            LinOpt xo;
            if (tc_o) xo.xs_in = M->xs_attn;
            x_ready = tc_o && linear_uses_tensor_cores(m, ff, d, true);
            if (x_ready) { xo.out_xs = M->xs_x; xo.out_ld = d; xo.out_gain = y.norm2; xo.out_ssq = M->ssq_x; }
            CSD_TRY(linear(M, y.xo, nullptr, d, di, M->attn, di, m, nullptr, M->x, d, EPI_ADD, st, &xo));
        }
        // feed-forward; its down projection hands the rows on to the next layer's first norm (or the final one)
        const bool last = l + 1 == c.n_layers;
        const __nv_bfloat16* next_gain = last ? M->final_norm : M->dec[l + 1].norm1;
        const LayerW* nx = last ? nullptr : &M->dec[l + 1];
        const bool fused_qkv = nx && nx->wk == nx->wq + (size_t)di * d && nx->wv == nx->wk + (size_t)di * d;
        const int next_N = last ? V : (fused_qkv ? 3 * di : di);
        CSD_TRY(feed_forward(M, y, M->x, m, st, x_ready, next_gain, next_N, false, &x_ready));
    }
    if (!logits_out_dev) {                    // cache append only: nobody reads this block's laws
        CSD_CUDA(cudaGetLastError());
        return CSD_OK;
    }
    LinOpt ho;
    if (x_ready) { ho.xs_in = M->xs_x; ho.ssq_in = M->ssq_x; ho.ssq_cnt = M->ssq_x_cnt; }
    CSD_TRY(linear(M, M->lm_head, nullptr, V, d, M->x, d, m, M->final_norm, logits_out_dev, V, EPI_STORE, st, &ho));
    CSD_CUDA(cudaGetLastError());
    return CSD_OK;
}
