// Review rule of speculative sampling (Section 2; lenience / greedy: Section 3.1) as three
// kernels over the vocabulary:
//   stats    one streaming pass over all (2k+1) logit vectors of every row: per 8192-logit piece
//            the max, arg-max and sum of exponentials (fp32).  This is the HBM-bound part: a
//            warp owns a piece, keeps 8 x 16 bytes per lane in flight with the next 8 already
//            requested, and needs no block-wide synchronisation.
//   decide   per row: merge the pieces, run the accept tests of all positions in parallel with
//            the Philox uniforms, find the first rejection n.
//   resample (temperature > 0 only) per row, at position n only, in fp64 so that the chosen token
//            does not depend on summation order or on fp32 rounding: first the per-chunk sums
//            of the exponentials (the normalisers), then per chunk the mass of the residual
//            max(0, p - q) (or of p after k acceptances); the CTA that finishes a row last takes
//            the inverse-CDF pick.  exp() here is a short fp64 routine of this file (argument
//            reduction by ln 2 and a degree-11 Taylor polynomial, relative error below 1e-13 on
//            the arguments that occur, x <= 0), and every division is a multiplication by a
//            reciprocal formed once.
#include "common.cuh"
#include "philox.cuh"
#include <math.h>
#include <mutex>

namespace csd {

constexpr int ST_THREADS = 256;
constexpr int ST_CHUNK = 8192;   // logits per warp item of the stats pass
constexpr int ST_SUB = 1024;     // logits a warp has in registers at a time (8 x float4 per lane)
constexpr int RS_THREADS = 256;
constexpr int RS_PER_THREAD = 8;
constexpr int RS_CHUNK = RS_THREADS * RS_PER_THREAD;  // logits per CTA of the resample pass

struct __align__(16) StatPartial {
    float mx;
    float sum;   // sum exp((x - mx) * invT) over the piece
    int arg;     // smallest index attaining mx
    int pad;
};

enum : int { MODE_DONE = 0, MODE_RESID_LOGITS = 1, MODE_RESID_POINT = 2, MODE_TARGET_ONLY = 3 };

struct __align__(16) RowInfo {
    int n;        // first rejected position (k if none)
    int mode;
    int x;        // drafted token at position n (point-mass / validation)
    int pad;
    double max_t; // max target logit at position n
    double max_q; // max draft logit at position n
    double u2;    // resampling uniform
};

// ---------------------------------------------------------------------------------------------
// stats pass: grid-stride loop of warps over (vector, piece) items
// ---------------------------------------------------------------------------------------------
template <bool VEC>
__device__ __forceinline__ void load_sub(const float* __restrict__ src, int e0, int V, int lane, float (&v)[32]) {
    if (VEC) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int e = e0 + 4 * (lane + 32 * j);
            float4 f = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
            if (e < V) f = __ldcs(reinterpret_cast<const float4*>(src + e));
            v[4 * j + 0] = f.x; v[4 * j + 1] = f.y; v[4 * j + 2] = f.z; v[4 * j + 3] = f.w;
        }
    } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            const int e = e0 + lane + 32 * j;
            v[j] = e < V ? __ldcs(src + e) : -INFINITY;
        }
    }
}
template <bool VEC> __device__ __forceinline__ int sub_index(int e0, int lane, int j) {
    return VEC ? e0 + 4 * (lane + 32 * (j >> 2)) + (j & 3) : e0 + lane + 32 * j;
}

template <bool VEC>
__global__ void __launch_bounds__(ST_THREADS, 2)
accept_stats_kernel(const float* __restrict__ tl, const float* __restrict__ dl, long long n_tvec, int V,
                    float invT, int greedy, StatPartial* __restrict__ out, int nchunk, long long items) {
    pdl_wait();            // the logits come from the kernel before this one on the stream
    pdl_trigger();
    const int lane = threadIdx.x & 31;
    const long long warps = (long long)gridDim.x * (ST_THREADS / 32);
    for (long long item = (long long)blockIdx.x * (ST_THREADS / 32) + (threadIdx.x >> 5); item < items; item += warps) {
        const long long vec = item / nchunk;
        const int chunk = (int)(item % nchunk);
        const float* src = vec < n_tvec ? tl + vec * (long long)V : dl + (vec - n_tvec) * (long long)V;
        const int base = chunk * ST_CHUNK;
        const int nsub = (min(V, base + ST_CHUNK) - base + ST_SUB - 1) / ST_SUB;
        float mx = -INFINITY, sum = 0.f;
        int arg = 0x7fffffff;
        float cur[32], nxt[32];
        load_sub<VEC>(src, base, V, lane, cur);
        for (int s = 0; s < nsub; ++s) {
            const int e0 = base + s * ST_SUB;
            if (s + 1 < nsub) load_sub<VEC>(src, e0 + ST_SUB, V, lane, nxt);     // in flight while this batch is reduced
            // batch max with the smallest index attaining it (indices grow with j inside a lane)
            float bm = -INFINITY;
            int ba = 0x7fffffff;
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (cur[j] > bm) { bm = cur[j]; ba = sub_index<VEC>(e0, lane, j); }
            if (bm > mx) {          // later batches hold larger indices, so ">" keeps the earliest arg-max
                sum = mx > -INFINITY ? sum * __expf((mx - bm) * invT) : 0.f;
                mx = bm; arg = ba;
            }
            if (!greedy && mx > -INFINITY) {
                float a = 0.f;
#pragma unroll
                for (int j = 0; j < 32; ++j) a += __expf((cur[j] - mx) * invT);
                sum += a;
            }
            if (s + 1 < nsub) {
#pragma unroll
                for (int j = 0; j < 32; ++j) cur[j] = nxt[j];
            }
        }
        // lanes -> warp
        float wm = mx;
        int wa = arg;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float om = __shfl_xor_sync(0xffffffffu, wm, o);
            const int oa = __shfl_xor_sync(0xffffffffu, wa, o);
            if (om > wm || (om == wm && oa < wa)) { wm = om; wa = oa; }
        }
        float scaled = (!greedy && mx > -INFINITY) ? sum * __expf((mx - wm) * invT) : 0.f;
        scaled = warp_sum(scaled);
        if (lane == 0) {
            StatPartial p;
            p.mx = wm; p.sum = scaled; p.arg = wa; p.pad = 0;
            out[item] = p;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// decide pass: one CTA per row
// ---------------------------------------------------------------------------------------------
constexpr int MAX_K = 64;

__global__ void __launch_bounds__(128)
accept_decide_kernel(const float* __restrict__ tl, const float* __restrict__ dl, const int* __restrict__ onehot,
                     const int* __restrict__ tokens, int rows, int k, int V, float temperature, float lenience,
                     uint64_t seed, uint64_t step, const StatPartial* __restrict__ part, int nchunk,
                     int* __restrict__ n_acc, int* __restrict__ out_tok, RowInfo* __restrict__ info,
                     unsigned* __restrict__ tickets, int* status) {
    pdl_wait();
    pdl_trigger();
    const int row = blockIdx.x;
    __shared__ float s_mx[2 * MAX_K + 1];
    __shared__ float s_z[2 * MAX_K + 1];
    __shared__ int s_arg[2 * MAX_K + 1];
    __shared__ int s_acc[MAX_K], s_x[MAX_K], s_point[MAX_K];
    __shared__ double s_u2[MAX_K];
    const bool greedy = temperature == 0.f;
    const float invT = greedy ? 1.f : 1.f / temperature;
    const int nvec_row = dl ? 2 * k + 1 : k + 1;
    const long long n_tvec = (long long)rows * (k + 1);
    // ---- merge the pieces of every vector of this row (one thread per vector, one pass)
    for (int i = threadIdx.x; i < nvec_row; i += blockDim.x) {
        const long long vec = i <= k ? (long long)row * (k + 1) + i : n_tvec + (long long)row * k + (i - k - 1);
        const StatPartial* p = part + vec * nchunk;
        float mx = -INFINITY, z = 0.f;
        int arg = 0x7fffffff;
#pragma unroll 4
        for (int c = 0; c < nchunk; ++c) {
            const StatPartial q = p[c];
            if (q.mx > mx) {        // pieces come in index order, so ">" keeps the earliest arg-max
                z = mx > -INFINITY ? z * __expf((mx - q.mx) * invT) : 0.f;
                mx = q.mx; arg = q.arg;
                z += q.sum;
            } else if (q.mx > -INFINITY) {
                z += q.sum * __expf((q.mx - mx) * invT);
            }
        }
        s_mx[i] = mx; s_z[i] = greedy ? 0.f : z; s_arg[i] = arg;
    }
    if (threadIdx.x == 0 && tickets) { tickets[row] = 0u; tickets[rows + row] = 0u; }   // for the two resample passes
    __syncthreads();
    const int* tok = tokens + (long long)row * k;
    RowInfo ri;
    ri.n = k; ri.mode = MODE_DONE; ri.x = 0; ri.pad = 0; ri.max_t = 0; ri.max_q = 0; ri.u2 = 0;
    if (greedy) {
        if (threadIdx.x != 0) return;
        int n = 0;
        while (n < k && tok[n] == s_arg[n]) ++n;
        for (int i = 0; i < k; ++i)             // a drafted id outside the vocabulary is rejected and recorded
            if (tok[i] < 0 || tok[i] >= V) set_status(status, CSD_ERR_BAD_TOKEN);
        n_acc[row] = n;
        out_tok[row] = s_arg[n];
        ri.n = n;
        info[row] = ri;
        return;
    }
    const uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
    const uint32_t c2 = (uint32_t)step, c3 = (uint32_t)(step >> 32);
    const double T = (double)temperature;
    // ---- the accept tests of all positions at once (thread i: position i)
    for (int i = threadIdx.x; i < k; i += blockDim.x) {
        int x = tok[i];
        const Philox4 r = philox4x32_10((uint32_t)i, (uint32_t)row, c2, c3, k0, k1);
        const bool point = dl == nullptr || (onehot && onehot[(long long)row * k + i] != 0);
        bool accept = false;
        if (x < 0 || x >= V) {
            set_status(status, CSD_ERR_BAD_TOKEN);
            x = 0;
        } else {
            const double u = word_uniform(r.w[0]);
            const double px = exp(((double)tl[((long long)row * (k + 1) + i) * V + x] - (double)s_mx[i]) / T) / (double)s_z[i];
            double qx = 1.0;
            if (!point)
                qx = exp(((double)dl[((long long)row * k + i) * V + x] - (double)s_mx[k + 1 + i]) / T) /
                     (double)s_z[k + 1 + i];
            accept = u * qx < (point ? 1.0 : (double)lenience) * px;   // no lenience for the statistical drafter's tokens (Appendix B)
        }
        s_acc[i] = accept ? 1 : 0; s_x[i] = x; s_point[i] = point ? 1 : 0; s_u2[i] = word_uniform(r.w[1]);
    }
    __syncthreads();
    if (threadIdx.x != 0) return;
    int n = 0;
    while (n < k && s_acc[n]) ++n;
    if (n < k) {
        const bool point = s_point[n] != 0;
        ri.mode = point ? MODE_RESID_POINT : MODE_RESID_LOGITS;
        ri.x = s_x[n];
        ri.max_t = (double)s_mx[n];
        ri.max_q = point ? 0.0 : (double)s_mx[k + 1 + n];
        ri.u2 = s_u2[n];
    } else {
        const Philox4 r = philox4x32_10((uint32_t)k, (uint32_t)row, c2, c3, k0, k1);
        ri.mode = MODE_TARGET_ONLY;
        ri.max_t = (double)s_mx[k];
        ri.u2 = word_uniform(r.w[1]);
    }
    ri.n = n;
    n_acc[row] = n;
    info[row] = ri;
}

// ---------------------------------------------------------------------------------------------
// resample passes (fp64).  grid = (rows, chunks).  Every sum has one fixed order: lanes by
// xor-shuffle, warps in index order, chunks in index order.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ double block_sum_ordered(double v, double* s_warp) {
    v = warp_sum(v);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) s_warp[warp] = v;
    __syncthreads();
    double tot = 0.0;
    for (int w = 0; w < RS_THREADS / 32; ++w) tot += s_warp[w];
    return tot;
}

// exp(x) for x <= 0 in fp64 by table and polynomial: x = (64 m + j) ln2/64 + r with |r| <= ln2/128,
// exp(x) = 2^m * 2^(j/64) * e^r; the 64 table entries are correctly rounded doubles made on the host,
// e^r is its Taylor series to r^5 (remainder below 4e-17), 2^m goes through the exponent field.
// Relative error about 3e-16.  Below -708 the result is 0 (under the smallest normal number).
__constant__ double c_exp2_table[64];
__device__ __forceinline__ void exp_table_to_shared(double* s_tab) {
    for (int i = threadIdx.x; i < 64; i += blockDim.x) s_tab[i] = c_exp2_table[i];
    __syncthreads();
}
__device__ __forceinline__ double exp_neg(double x, const double* __restrict__ s_tab) {
    if (!(x > -708.0)) return 0.0;
    const double nf = rint(x * 92.33248261689366);           // 64 / ln 2
    double r = fma(-nf, 0.01083042468962958, x);              // ln 2 / 64, high part (low 22 bits clear: nf * high is exact)
    r = fma(-nf, 6.619564634077006e-12, r);                   // ln 2 / 64, low part
    const int n = (int)nf;
    double p = 1.0 / 120.0;
    p = fma(p, r, 1.0 / 24.0);
    p = fma(p, r, 1.0 / 6.0);
    p = fma(p, r, 0.5);
    p = fma(p, r, 1.0);
    p *= r;                                                   // e^r - 1
    const double tj = s_tab[n & 63];
    const double v = fma(tj, p, tj);
    const long long bits = __double_as_longlong(v) + ((long long)(n >> 6) << 52);   // m >= -1022: stays a normal number
    return __longlong_as_double(bits);
}

// eight consecutive logits of a vector (two 16-byte loads when the vector allows it); past V: -inf
__device__ __forceinline__ void load8(const float* __restrict__ src, int e0, int V, bool vec, float (&v)[8]) {
    if (vec && e0 + 7 < V) {
        const float4 a = __ldcs(reinterpret_cast<const float4*>(src + e0));
        const float4 b = __ldcs(reinterpret_cast<const float4*>(src + e0 + 4));
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = e0 + j < V ? __ldcs(src + e0 + j) : -INFINITY;
    }
}

struct ResidualCtx {
    const float* t; const float* d; const double* tab;
    double max_t, max_q, invT, inv_zt, inv_zq;
    int mode, x;
};
__device__ __forceinline__ double residual_at(const ResidualCtx& c, int e) {
    const double p = exp_neg(((double)c.t[e] - c.max_t) * c.invT, c.tab) * c.inv_zt;
    if (c.mode == MODE_TARGET_ONLY) return p;
    const double q = c.mode == MODE_RESID_POINT ? (e == c.x ? 1.0 : 0.0)
                                                : exp_neg(((double)c.d[e] - c.max_q) * c.invT, c.tab) * c.inv_zq;
    const double r = p - q;
    return r > 0.0 ? r : 0.0;
}

__device__ __forceinline__ double residual_of(const ResidualCtx& c, int e, float tv, float dv) {
    const double p = exp_neg(((double)tv - c.max_t) * c.invT, c.tab) * c.inv_zt;
    if (c.mode == MODE_TARGET_ONLY) return p;
    const double q = c.mode == MODE_RESID_POINT ? (e == c.x ? 1.0 : 0.0)
                                                : exp_neg(((double)dv - c.max_q) * c.invT, c.tab) * c.inv_zq;
    const double r = p - q;
    return r > 0.0 ? r : 0.0;
}

// pass 1: per-chunk sums of exp((t - max_t)/T) and exp((d - max_q)/T)
__global__ void __launch_bounds__(RS_THREADS)
resample_z_kernel(const float* __restrict__ tl, const float* __restrict__ dl, int k, int V, float temperature,
                  const RowInfo* __restrict__ info, double2* __restrict__ zpart, double2* __restrict__ zsum,
                  unsigned* __restrict__ tickets, int nchunk) {
    const int row = blockIdx.x, chunk = blockIdx.y;
    __shared__ double s_warp[RS_THREADS / 32];
    __shared__ double s_tab[64];
    exp_table_to_shared(s_tab);
    pdl_wait();            // the row records come from the decide pass
    pdl_trigger();
    const RowInfo ri = info[row];
    if (ri.mode == MODE_DONE) return;
    const double invT = 1.0 / (double)temperature;
    const float* t = tl + ((long long)row * (k + 1) + ri.n) * V;
    const float* d = ri.mode == MODE_RESID_LOGITS ? dl + ((long long)row * k + ri.n) * V : nullptr;
    const int e0 = chunk * RS_CHUNK + threadIdx.x * RS_PER_THREAD;
    double sp = 0.0, sq = 0.0;
    {
        static_assert(RS_PER_THREAD == 8, "load8 covers a thread's entries");
        const bool vec = (V % 4 == 0) && ((((uintptr_t)t) & 15) == 0) && (!d || (((uintptr_t)d) & 15) == 0);
        float tv[8], dv[8];
        load8(t, e0, V, vec, tv);
        if (d) load8(d, e0, V, vec, dv);
#pragma unroll
        for (int j = 0; j < RS_PER_THREAD; ++j) {
            sp += exp_neg(((double)tv[j] - ri.max_t) * invT, s_tab);      // -inf (past V) gives 0
            if (d) sq += exp_neg(((double)dv[j] - ri.max_q) * invT, s_tab);
        }
    }
    sp = block_sum_ordered(sp, s_warp);
    sq = block_sum_ordered(sq, s_warp);
    __shared__ int s_is_last;
    __shared__ double2 s_z[RS_THREADS];
    double2* zrow = zpart + (long long)row * nchunk;
    if (threadIdx.x == 0) {
        zrow[chunk] = make_double2(sp, sq);
        __threadfence();
        s_is_last = atomicAdd(&tickets[row], 1u) == (unsigned)nchunk - 1u;
    }
    __syncthreads();
    if (!s_is_last) return;
    // last chunk of the row: the totals, summed in chunk order (loads in parallel, adds by one thread)
    __threadfence();
    double Zp = 0.0, Zq = 0.0;
    for (int c0 = 0; c0 < nchunk; c0 += RS_THREADS) {
        const int c = c0 + threadIdx.x;
        s_z[threadIdx.x] = c < nchunk ? make_double2(__ldcg(&zrow[c].x), __ldcg(&zrow[c].y)) : make_double2(0.0, 0.0);
        __syncthreads();
        if (threadIdx.x == 0)
            for (int i = 0; i < RS_THREADS && c0 + i < nchunk; ++i) { Zp += s_z[i].x; Zq += s_z[i].y; }
        __syncthreads();
    }
    if (threadIdx.x == 0) zsum[row] = make_double2(Zp, Zq);
}

// pass 2: per-chunk mass of the residual; the CTA that arrives last at the row's ticket picks the token
__global__ void __launch_bounds__(RS_THREADS)
resample_pick_kernel(const float* __restrict__ tl, const float* __restrict__ dl, int k, int V, float temperature,
                     const RowInfo* __restrict__ info, const double2* __restrict__ zpart,
                     const double2* __restrict__ zsum, double* __restrict__ rpart, unsigned* __restrict__ tickets,
                     int nchunk, int* __restrict__ out_tok) {
    const int row = blockIdx.x, chunk = blockIdx.y;
    pdl_wait();            // the normalisers come from the pass before this one
    pdl_trigger();
    const RowInfo ri = info[row];
    if (ri.mode == MODE_DONE) return;
    __shared__ double s_warp[RS_THREADS / 32];
    __shared__ double s_scan[RS_THREADS / 32];
    __shared__ double s_d[2];    // target, base
    __shared__ int s_i[3];       // chunk, mode, forced-last flag
    __shared__ int s_pick, s_last, s_is_last;
    __shared__ double s_tab[64];
    exp_table_to_shared(s_tab);
    const double2* zrow = zpart + (long long)row * nchunk;
    double* rrow = rpart + (long long)row * nchunk;
    const double Zp = zsum[row].x, Zq = zsum[row].y;
    ResidualCtx c;
    c.t = tl + ((long long)row * (k + 1) + ri.n) * V;
    c.d = ri.mode == MODE_RESID_LOGITS ? dl + ((long long)row * k + ri.n) * V : nullptr;
    c.max_t = ri.max_t; c.max_q = ri.max_q; c.invT = 1.0 / (double)temperature;
    c.inv_zt = 1.0 / Zp; c.inv_zq = Zq > 0.0 ? 1.0 / Zq : 0.0;
    c.mode = ri.mode; c.x = ri.x; c.tab = s_tab;
    {
        const int e0 = chunk * RS_CHUNK + threadIdx.x * RS_PER_THREAD;
        const bool vec = (V % 4 == 0) && ((((uintptr_t)c.t) & 15) == 0) && (!c.d || (((uintptr_t)c.d) & 15) == 0);
        float tv[8], dv[8];
        load8(c.t, e0, V, vec, tv);
        if (c.d) load8(c.d, e0, V, vec, dv);
        double sr = 0.0;
#pragma unroll
        for (int j = 0; j < RS_PER_THREAD; ++j)
            if (e0 + j < V) sr += residual_of(c, e0 + j, tv[j], c.d ? dv[j] : 0.f);
        sr = block_sum_ordered(sr, s_warp);
        if (threadIdx.x == 0) {
            rrow[chunk] = sr;
            __threadfence();
            s_is_last = atomicAdd(&tickets[row], 1u) == (unsigned)nchunk - 1u;
        }
        __syncthreads();
        if (!s_is_last) return;
        __threadfence();
    }
    // ---- last CTA of the row: which chunk holds u2 * S, then the entry inside it.  Chunk masses are
    //      fetched by all threads into shared memory; one thread adds them in chunk order.
    __shared__ double s_mass[RS_THREADS];
    __shared__ double s_S;
    __shared__ int s_empty;
    for (int pass = 0; pass < 2; ++pass) {
        // pass 0: total mass S (and whether the residual is empty); pass 1: the chunk that holds u2 * S
        const bool empty = pass == 1 && s_empty;
        double acc = 0.0, target = 0.0;
        int pick_chunk = -1, last_pos = 0;
        double base = 0.0;
        if (pass == 1) target = ri.u2 * s_S;
        for (int c0 = 0; c0 < nchunk; c0 += RS_THREADS) {
            const int ch = c0 + threadIdx.x;
            double mval = 0.0;
            if (ch < nchunk) mval = empty ? zrow[ch].x * c.inv_zt : __ldcg(rrow + ch);
            s_mass[threadIdx.x] = mval;
            __syncthreads();
            if (threadIdx.x == 0) {
                for (int i = 0; i < RS_THREADS && c0 + i < nchunk; ++i) {
                    const double mass = s_mass[i];
                    if (pass == 0) { acc += mass; continue; }
                    if (pick_chunk >= 0) break;
                    if (mass > 0.0) last_pos = c0 + i;
                    if (acc + mass > target) { pick_chunk = c0 + i; base = acc; break; }
                    acc += mass;
                }
            }
            __syncthreads();
        }
        if (threadIdx.x == 0) {
            if (pass == 0) {
                const bool is_empty = !(acc > 0.0) || !isfinite(acc);
                s_empty = is_empty ? 1 : 0;
                if (is_empty) {   // empty residual: fall back to the target law itself
                    acc = 0.0;
                    for (int ch = 0; ch < nchunk; ++ch) acc += zrow[ch].x * c.inv_zt;
                }
                s_S = acc;
            } else {
                int forced = 0;
                if (pick_chunk < 0) { pick_chunk = last_pos; forced = 1; }
                s_d[0] = target; s_d[1] = base;
                s_i[0] = pick_chunk; s_i[1] = s_empty ? (int)MODE_TARGET_ONLY : ri.mode; s_i[2] = forced;
                s_pick = 0x7fffffff; s_last = -1;
            }
        }
        __syncthreads();
    }
    const double target = s_d[0], base = s_d[1];
    const int pick_chunk = s_i[0], forced = s_i[2];
    c.mode = s_i[1];
    const int e0 = pick_chunk * RS_CHUNK + threadIdx.x * RS_PER_THREAD;
    double r[RS_PER_THREAD];
    double local = 0.0;
    int my_last = -1;
#pragma unroll
    for (int j = 0; j < RS_PER_THREAD; ++j) {
        const int e = e0 + j;
        r[j] = 0.0;
        if (e < V) {
            r[j] = residual_at(c, e);
            if (r[j] > 0.0) my_last = e;
        }
        local += r[j];
    }
    // exclusive prefix of the per-thread sums, in thread order
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    double incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) s_scan[warp] = incl;
    __syncthreads();
    double woff = 0.0;
    for (int w = 0; w < warp; ++w) woff += s_scan[w];
    double cum = base + woff + (incl - local);
    int found = 0x7fffffff;
    if (!forced) {
#pragma unroll
        for (int j = 0; j < RS_PER_THREAD; ++j) {
            cum += r[j];
            if (found == 0x7fffffff && r[j] > 0.0 && cum > target) found = e0 + j;
        }
    }
    if (found != 0x7fffffff) atomicMin(&s_pick, found);
    if (my_last >= 0) atomicMax(&s_last, my_last);
    __syncthreads();
    if (threadIdx.x == 0) out_tok[row] = s_pick != 0x7fffffff ? s_pick : (s_last >= 0 ? s_last : 0);
}

// ---------------------------------------------------------------------------------------------
// resample, one kernel: a row is a thread-block cluster of up to RF_MAXC CTAs; a CTA keeps its
// slice of the two logit vectors (position n only) in registers, so global memory is read once.
// First exchange: per-CTA sums of the exponentials, exchanged through distributed shared memory -> the
// normalisers.  Second exchange: per-CTA residual mass -> total mass S and the CTA whose slice holds
// u2 * S.  That CTA scans its threads' sums in thread order and picks the entry.  All sums have a
// fixed order (lanes by xor-shuffle or prefix scan, warps and CTAs in index order).
// ---------------------------------------------------------------------------------------------
constexpr int RF_THREADS = 512, RF_PER = 16, RF_SLICE = RF_THREADS * RF_PER, RF_MAXC = 16;
constexpr int RF_USE_MAXC = 8;   // larger clusters run (one per GPC at a time) but lose to the two-pass kernels: 199 us against 145 at V = 128256

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ double cluster_read_f64(const double* local, uint32_t rank) {
    uint32_t a = (uint32_t)__cvta_generic_to_shared(local), r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(rank));
    double v;
    asm volatile("ld.shared::cluster.f64 %0, [%1];" : "=d"(v) : "r"(r) : "memory");
    return v;
}

// ordered sum over the CTA; the result is valid in every thread
__device__ __forceinline__ double rf_block_sum(double v, double* s_warp) {
    v = warp_sum(v);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) s_warp[warp] = v;
    __syncthreads();
    double tot = 0.0;
    for (int w = 0; w < RF_THREADS / 32; ++w) tot += s_warp[w];
    return tot;
}

__global__ void __launch_bounds__(RF_THREADS, 1)
resample_fused_kernel(const float* __restrict__ tl, const float* __restrict__ dl, int k, int V, float temperature,
                      const RowInfo* __restrict__ info, int csize, int* __restrict__ out_tok) {
    const int row = blockIdx.x / csize;
    const uint32_t rank = cluster_rank();
    pdl_wait();            // the row records come from the decide pass
    pdl_trigger();
    const RowInfo ri = info[row];
    if (ri.mode == MODE_DONE) return;                 // (the same decision in every CTA of the cluster)
    __shared__ double s_warp[RF_THREADS / 32];
    __shared__ double s_ex[2];                        // this CTA's contribution to the current exchange
    __shared__ double s_scan[RF_THREADS / 32];
    __shared__ int s_pick, s_last;
    __shared__ double s_tab[64];
    exp_table_to_shared(s_tab);
    const double invT = 1.0 / (double)temperature;
    const float* t = tl + ((long long)row * (k + 1) + ri.n) * V;
    const float* d = ri.mode == MODE_RESID_LOGITS ? dl + ((long long)row * k + ri.n) * V : nullptr;
    const int e0 = (int)rank * RF_SLICE + threadIdx.x * RF_PER;
    // ---- this thread's entries, read once; their exponentials stay in registers for both rounds
    double et[RF_PER], ed[RF_PER];
    const bool vec = (V % 4 == 0) && ((((uintptr_t)t) & 15) == 0) && (!d || (((uintptr_t)d) & 15) == 0);
    double sp = 0.0, sq = 0.0;
#pragma unroll
    for (int j = 0; j < RF_PER; j += 4) {
        const int e = e0 + j;
        float tv[4], dv[4];
        if (vec && e + 3 < V) {
            const float4 a = __ldcs(reinterpret_cast<const float4*>(t + e));
            tv[0] = a.x; tv[1] = a.y; tv[2] = a.z; tv[3] = a.w;
            if (d) {
                const float4 b = __ldcs(reinterpret_cast<const float4*>(d + e));
                dv[0] = b.x; dv[1] = b.y; dv[2] = b.z; dv[3] = b.w;
            } else { dv[0] = dv[1] = dv[2] = dv[3] = -INFINITY; }
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                tv[i] = e + i < V ? __ldcs(t + e + i) : -INFINITY;
                dv[i] = (d && e + i < V) ? __ldcs(d + e + i) : -INFINITY;
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            et[j + i] = exp_neg(((double)tv[i] - ri.max_t) * invT, s_tab);   // -inf (past V) gives 0
            ed[j + i] = d ? exp_neg(((double)dv[i] - ri.max_q) * invT, s_tab) : 0.0;
            sp += et[j + i];
            sq += ed[j + i];
        }
    }
    // ---- first exchange: normalisers
    sp = rf_block_sum(sp, s_warp);
    sq = rf_block_sum(sq, s_warp);
    if (threadIdx.x == 0) { s_ex[0] = sp; s_ex[1] = sq; }
    cluster_sync_all();
    double Zp = 0.0, Zq = 0.0;
    for (int c = 0; c < csize; ++c) { Zp += cluster_read_f64(&s_ex[0], (uint32_t)c); Zq += cluster_read_f64(&s_ex[1], (uint32_t)c); }
    cluster_sync_all();                               // everyone has read before s_ex is reused
    ResidualCtx cx;
    cx.t = nullptr; cx.d = nullptr; cx.tab = s_tab; cx.max_t = ri.max_t; cx.max_q = ri.max_q; cx.invT = invT;
    cx.inv_zt = 1.0 / Zp; cx.inv_zq = Zq > 0.0 ? 1.0 / Zq : 0.0; cx.mode = ri.mode; cx.x = ri.x;
    auto resid = [&](int j, int mode) -> double {
        if (e0 + j >= V) return 0.0;
        const double p = et[j] * cx.inv_zt;
        if (mode == MODE_TARGET_ONLY) return p;
        const double q = mode == MODE_RESID_POINT ? (e0 + j == cx.x ? 1.0 : 0.0) : ed[j] * cx.inv_zq;
        const double r = p - q;
        return r > 0.0 ? r : 0.0;
    };
    // ---- second exchange: masses (a second time with the target law itself if the residual is empty)
    int mode = ri.mode;
    double local = 0.0, S = 0.0, base = 0.0, my_mass = 0.0;
    int pick_cta = -1, last_pos = 0;
    for (int pass = 0; pass < 2; ++pass) {
        local = 0.0;
#pragma unroll
        for (int j = 0; j < RF_PER; ++j) local += resid(j, mode);
        my_mass = rf_block_sum(local, s_warp);
        if (threadIdx.x == 0) s_ex[0] = my_mass;
        cluster_sync_all();
        S = 0.0;
        double masses[RF_MAXC];
        for (int c = 0; c < csize; ++c) { masses[c] = cluster_read_f64(&s_ex[0], (uint32_t)c); S += masses[c]; }
        cluster_sync_all();
        const bool empty = !(S > 0.0) || !isfinite(S);
        if (empty && pass == 0 && mode != MODE_TARGET_ONLY) { mode = MODE_TARGET_ONLY; continue; }
        const double target = ri.u2 * S;
        double acc = 0.0;
        for (int c = 0; c < csize; ++c) {
            if (masses[c] > 0.0) last_pos = c;
            if (pick_cta < 0 && acc + masses[c] > target) { pick_cta = c; base = acc; }
            if (pick_cta < 0) acc += masses[c];
        }
        break;
    }
    const double target = ri.u2 * S;
    int forced = 0;
    if (pick_cta < 0) { pick_cta = last_pos; forced = 1; }
    if ((int)rank != pick_cta) return;
    // ---- the picking CTA: exclusive prefix of the threads' sums in thread order, then the entry
    if (threadIdx.x == 0) { s_pick = 0x7fffffff; s_last = -1; }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    double incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) s_scan[warp] = incl;
    __syncthreads();
    double woff = 0.0;
    for (int w = 0; w < warp; ++w) woff += s_scan[w];
    double cum = base + woff + (incl - local);
    int found = 0x7fffffff, my_last = -1;
#pragma unroll
    for (int j = 0; j < RF_PER; ++j) {
        const double r = resid(j, mode);
        if (r > 0.0) my_last = e0 + j;
        cum += r;
        if (!forced && found == 0x7fffffff && r > 0.0 && cum > target) found = e0 + j;
    }
    if (found != 0x7fffffff) atomicMin(&s_pick, found);
    if (my_last >= 0) atomicMax(&s_last, my_last);
    __syncthreads();
    if (threadIdx.x == 0) out_tok[row] = s_pick != 0x7fffffff ? s_pick : (s_last >= 0 ? s_last : 0);
}

struct AcceptLayout {
    size_t part_off, info_off, z_off, zsum_off, r_off, ticket_off, total;
    int nchunk_a, nchunk_r;
};

static AcceptLayout accept_layout(int rows, int k, int V) {
    AcceptLayout L;
    L.nchunk_a = (V + ST_CHUNK - 1) / ST_CHUNK;
    L.nchunk_r = (V + RS_CHUNK - 1) / RS_CHUNK;
    size_t nvec = (size_t)rows * (2 * (size_t)k + 1);
    size_t off = 0;
    L.part_off = off;   off = align_up(off + nvec * L.nchunk_a * sizeof(StatPartial), 256);
    L.info_off = off;   off = align_up(off + (size_t)rows * sizeof(RowInfo), 256);
    L.z_off = off;      off = align_up(off + (size_t)rows * L.nchunk_r * sizeof(double2), 256);
    L.r_off = off;      off = align_up(off + (size_t)rows * L.nchunk_r * sizeof(double), 256);
    L.zsum_off = off;   off = align_up(off + (size_t)rows * sizeof(double2), 256);
    L.ticket_off = off; off = align_up(off + 2 * (size_t)rows * sizeof(unsigned), 256);   // normaliser pass, mass pass
    L.total = off;
    return L;
}

static int accept_sm_count() {
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
    }
    return n;
}

// The table of 2^(j/64), correctly rounded, goes to constant memory once per device.
static csd_status exp_table_ready() {
    static bool done[64];
    static std::mutex mu;
    int dev = 0;
    CSD_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return CSD_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(mu);
    if (!done[dev]) {
        double tab[64];
        for (int j = 0; j < 64; ++j) tab[j] = exp2((double)j / 64.0);
        CSD_CUDA(cudaMemcpyToSymbol(c_exp2_table, tab, sizeof(tab)));
        done[dev] = true;
    }
    return CSD_OK;
}

// Whether clusters of `csize` CTAs of the fused resample kernel can run on this device (sizes above
// 8 are an opt-in of the hardware); asked once per size.
static bool fused_resample_ok(int csize) {
    static int state[RF_MAXC + 1];              // 0 unknown, 1 yes, 2 no
    if (csize < 1 || csize > RF_USE_MAXC) return false;
    if (state[csize] == 0) {
        bool ok = true;
        if (csize > 8)
            ok = cudaFuncSetAttribute(resample_fused_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess;
        if (ok) {
            cudaLaunchConfig_t cfg = cudaLaunchConfig_t{};
            cudaLaunchAttribute attr[1];
            cfg.gridDim = dim3((unsigned)csize); cfg.blockDim = dim3(RF_THREADS);
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = (unsigned)csize; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr; cfg.numAttrs = 1;
            int n = 0;
            ok = cudaOccupancyMaxActiveClusters(&n, resample_fused_kernel, &cfg) == cudaSuccess && n >= 1;
        }
        if (!ok) (void)cudaGetLastError();
        state[csize] = ok ? 1 : 2;
    }
    return state[csize] == 1;
}

// The three passes on scratch `ws` (accept_layout bytes).  Every word a pass reads is written by an
// earlier pass of the same call (the decide pass clears the resample tickets), so the scratch
// needs no initialisation.
static csd_status run_accept(const float* tl, const float* dl_in, const int32_t* onehot, const int32_t* tokens, int rows,
                             int k, int V, float temperature, float lenience, uint64_t seed, uint64_t step,
                             int32_t* n_acc, int32_t* out_tok, char* ws, const AcceptLayout& L, int* status,
                             cudaStream_t st) {
    StatPartial* part = (StatPartial*)(ws + L.part_off);
    RowInfo* info = (RowInfo*)(ws + L.info_off);
    double2* zpart = (double2*)(ws + L.z_off);
    double* rpart = (double*)(ws + L.r_off);
    double2* zsum = (double2*)(ws + L.zsum_off);
    unsigned* tickets = (unsigned*)(ws + L.ticket_off);
    const bool greedy = temperature == 0.f;
    const float invT = greedy ? 1.f : 1.f / temperature;
    const bool use_d = dl_in != nullptr && k > 0 && !greedy;
    const float* dl = use_d ? dl_in : nullptr;
    const long long n_tvec = (long long)rows * (k + 1);
    const long long nvec = n_tvec + (use_d ? (long long)rows * k : 0);
    if (nvec > 0x7fffffffLL) return CSD_ERR_UNSUPPORTED;
    const bool vec_ok = (V % 4 == 0) && (((uintptr_t)tl & 15) == 0) && (!use_d || ((uintptr_t)dl & 15) == 0);
    const long long items = nvec * L.nchunk_a;
    long long ctas = (items + ST_THREADS / 32 - 1) / (ST_THREADS / 32);
    const long long cap = (long long)accept_sm_count() * 2;       // two resident CTAs per SM, grid-stride beyond
    if (ctas > cap) ctas = cap;
    // both launched with programmatic stream serialisation: they are resident and waiting when their
    // predecessor retires (in the cascade that is the output head of the review forward)
    {
        PdlLaunch ls(dim3((unsigned)ctas), dim3(ST_THREADS), 0, st);
        const int greedy_i = greedy ? 1 : 0;
        if (vec_ok)
            CSD_CUDA(cudaLaunchKernelEx(&ls.cfg, accept_stats_kernel<true>, tl, dl, n_tvec, V, invT, greedy_i, part, L.nchunk_a, items));
        else
            CSD_CUDA(cudaLaunchKernelEx(&ls.cfg, accept_stats_kernel<false>, tl, dl, n_tvec, V, invT, greedy_i, part, L.nchunk_a, items));
        PdlLaunch ld(dim3((unsigned)rows), dim3(128), 0, st);
        CSD_CUDA(cudaLaunchKernelEx(&ld.cfg, accept_decide_kernel, tl, dl, (const int*)onehot, (const int*)tokens, rows, k, V,
                                    temperature, lenience, seed, step, (const StatPartial*)part, L.nchunk_a, (int*)n_acc,
                                    (int*)out_tok, info, tickets, status));
    }
    count_launch(2);
    const int csize = (V + RF_SLICE - 1) / RF_SLICE;
    if (!greedy) {
        const csd_status ts = exp_table_ready();
        if (ts != CSD_OK) return ts;
    }
    if (!greedy && fused_resample_ok(csize)) {  // a row fits one cluster: the fused resample kernel
        cudaLaunchConfig_t cfg = cudaLaunchConfig_t{};
        cudaLaunchAttribute attr[2];
        cfg.gridDim = dim3((unsigned)(rows * csize)); cfg.blockDim = dim3(RF_THREADS); cfg.dynamicSmemBytes = 0; cfg.stream = st;
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)csize; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = 2;
        CSD_CUDA(cudaLaunchKernelEx(&cfg, resample_fused_kernel, tl, dl, k, V, temperature, (const RowInfo*)info, csize,
                                    (int*)out_tok));
        count_launch();
    } else if (!greedy) {
        dim3 g2((unsigned)rows, (unsigned)L.nchunk_r);
        PdlLaunch lz(g2, dim3(RS_THREADS), 0, st);
        CSD_CUDA(cudaLaunchKernelEx(&lz.cfg, resample_z_kernel, tl, dl, k, V, temperature, (const RowInfo*)info, zpart, zsum, tickets,
                                    L.nchunk_r));
        PdlLaunch lp(g2, dim3(RS_THREADS), 0, st);
        CSD_CUDA(cudaLaunchKernelEx(&lp.cfg, resample_pick_kernel, tl, dl, k, V, temperature, (const RowInfo*)info,
                                    (const double2*)zpart, (const double2*)zsum, rpart, tickets + rows, L.nchunk_r, (int*)out_tok));
        count_launch(2);
    }
    CSD_CUDA(cudaGetLastError());
    return CSD_OK;
}

}  // namespace csd

using namespace csd;

extern "C" size_t csd_spec_accept_workspace_bytes(int rows, int k, int V) {
    if (rows < 0 || k < 0 || V < 1) return 0;
    return accept_layout(rows, k, V).total;
}

extern "C" csd_status csd_spec_accept(const float* target_logits_dev, const float* draft_logits_dev,
                                      const int32_t* onehot_dev, const int32_t* draft_tokens_dev, int rows, int k,
                                      int V, float temperature, float lenience, uint64_t seed, uint64_t step,
                                      int32_t* n_accepted_dev, int32_t* out_token_dev, void* workspace_dev,
                                      size_t workspace_bytes, void* stream) {
    if (rows < 0 || k < 0 || k > MAX_K || V < 1 || !(temperature >= 0.f) || !(lenience >= 1.f))
        return CSD_ERR_INVALID_ARG;
    if (rows == 0) return CSD_OK;
    if (!target_logits_dev || !n_accepted_dev || !out_token_dev || !workspace_dev) return CSD_ERR_INVALID_ARG;
    if (k > 0 && !draft_tokens_dev) return CSD_ERR_INVALID_ARG;
    if (((uintptr_t)workspace_dev & 255) != 0) return CSD_ERR_INVALID_ARG;
    const AcceptLayout L = accept_layout(rows, k, V);
    if (workspace_bytes < L.total) return CSD_ERR_CAPACITY;
    if (L.nchunk_r > 65535) return CSD_ERR_UNSUPPORTED;
    int* status = status_word_device();
    if (!status) return CSD_ERR_CUDA;
    return run_accept(target_logits_dev, draft_logits_dev, onehot_dev, draft_tokens_dev, rows, k, V, temperature, lenience,
                      seed, step, n_accepted_dev, out_token_dev, (char*)workspace_dev, L, status, (cudaStream_t)stream);
}


// ---------------------------------------------------------------------------------------------
// Greedy acceptance along a tree of drafted tokens (tree attention, Section 5.1 / Appendix B).
// ---------------------------------------------------------------------------------------------
namespace csd {

struct TreeShape { int parent[CSD_MAX_ROWS]; };

// arg-max of every row of the target logits (smallest index on ties), one CTA per row
__global__ void __launch_bounds__(256)
tree_argmax_kernel(const float* __restrict__ logits, int V, int* __restrict__ arg) {
    pdl_wait();
    pdl_trigger();
    const float* x = logits + (size_t)blockIdx.x * V;
    float best = -INFINITY;
    int at = 0x7fffffff;
    for (int i = threadIdx.x; i < V; i += 256) {
        const float v = x[i];
        if (v > best || at == 0x7fffffff) { best = v; at = i; }
    }
    __shared__ float s_v[256];
    __shared__ int s_i[256];
    s_v[threadIdx.x] = best; s_i[threadIdx.x] = at;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) {
            const float ov = s_v[threadIdx.x + o];
            const int oi = s_i[threadIdx.x + o];
            if (ov > s_v[threadIdx.x] || (ov == s_v[threadIdx.x] && oi < s_i[threadIdx.x])) { s_v[threadIdx.x] = ov; s_i[threadIdx.x] = oi; }
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) arg[blockIdx.x] = s_i[0] == 0x7fffffff ? 0 : s_i[0];
}

// out[0] = tokens emitted, out[1] = leading rows of the accepted path that are a chain 0, 1, 2, ..
// (their cache entries are valid), out[2 ..] = the emitted tokens, out[2 + m ..] = rows of the path
__global__ void tree_walk_kernel(const int* __restrict__ arg, const int* __restrict__ tokens, const TreeShape shape, int m,
                                 int V, int* __restrict__ out, int* status) {
    if (threadIdx.x != 0) return;
    int cur = 0, n_out = 0, n_valid = 1;
    bool chain = true;
    out[2 + m] = 0;
    while (true) {
        const int y = arg[cur];
        out[2 + n_out] = y;
        ++n_out;
        int nxt = -1;
        for (int c = cur + 1; c < m; ++c) {
            const int t = tokens[c];
            if (t < 0 || t >= V) { set_status(status, CSD_ERR_BAD_TOKEN); continue; }
            if (shape.parent[c] == cur && t == y) { nxt = c; break; }
        }
        if (nxt < 0 || n_out >= m) break;
        out[2 + m + n_out] = nxt;
        chain = chain && nxt == n_out;
        if (chain) n_valid = n_out + 1;
        cur = nxt;
    }
    out[0] = n_out;
    out[1] = n_valid;
}

}  // namespace csd

extern "C" csd_status csd_tree_accept_greedy(const float* target_logits_dev, const int32_t* tokens_dev,
                                             const int32_t* parent_host, int n_rows, int V, int32_t* out_dev, void* stream) {
    if (!target_logits_dev || !tokens_dev || !parent_host || !out_dev || n_rows < 1 || n_rows > CSD_MAX_ROWS || V < 1)
        return CSD_ERR_INVALID_ARG;
    TreeShape shape;
    for (int r = 0; r < CSD_MAX_ROWS; ++r) shape.parent[r] = -2;
    for (int r = 0; r < n_rows; ++r) {
        const int p = parent_host[r];
        if (r == 0 ? p != -1 : (p < 0 || p >= r)) return CSD_ERR_INVALID_ARG;
        shape.parent[r] = p;
    }
    int* status = status_word_device();
    if (!status) return CSD_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    int* arg = (int*)out_dev + 2 + 2 * n_rows;
    PdlLaunch la(dim3((unsigned)n_rows), dim3(256), 0, st);
    CSD_CUDA(cudaLaunchKernelEx(&la.cfg, tree_argmax_kernel, target_logits_dev, V, arg));
    tree_walk_kernel<<<1, 32, 0, st>>>((const int*)arg, (const int*)tokens_dev, shape, n_rows, V, (int*)out_dev, status);
    count_launch(2);
    CSD_CUDA(cudaGetLastError());
    return CSD_OK;
}

// ---------------------------------------------------------------------------------------------
// Variant for callers that must not allocate: its scratch is a fixed array inside the library.
// ---------------------------------------------------------------------------------------------
namespace csd {
constexpr size_t STATIC_SCRATCH_BYTES = (size_t)2 << 20;   // 2 MiB, held by every GPU that loads the library
static __device__ __align__(256) unsigned char g_accept_scratch[STATIC_SCRATCH_BYTES];
constexpr int MAX_DEVICES = 64;
static void* g_accept_scratch_ptr[MAX_DEVICES];             // device address of the array, per device
static std::mutex g_accept_scratch_mu;
}  // namespace csd

extern "C" size_t csd_spec_accept_static_capacity(void) { return STATIC_SCRATCH_BYTES; }

extern "C" csd_status csd_spec_accept_static(const float* target_logits_dev, const float* draft_logits_dev,
                                             const int32_t* onehot_dev, const int32_t* draft_tokens_dev, int rows,
                                             int k, int V, float temperature, float lenience, uint64_t seed,
                                             uint64_t step, int32_t* n_accepted_dev, int32_t* out_token_dev,
                                             void* stream) {
    if (rows < 0 || k < 0 || k > MAX_K || V < 1 || !(temperature >= 0.f) || !(lenience >= 1.f))
        return CSD_ERR_INVALID_ARG;
    if (rows == 0) return CSD_OK;
    if (!target_logits_dev || !n_accepted_dev || !out_token_dev) return CSD_ERR_INVALID_ARG;
    if (k > 0 && !draft_tokens_dev) return CSD_ERR_INVALID_ARG;
    const AcceptLayout L = accept_layout(rows, k, V);
    if (L.total > STATIC_SCRATCH_BYTES) return CSD_ERR_CAPACITY;   // the problem does not fit the fixed scratch
    if (L.nchunk_r > 65535) return CSD_ERR_UNSUPPORTED;
    // Set-up, once per device: in host code the array's name is only a handle, so ask the runtime
    // for the address the kernels can use.  Nothing is allocated here.
    int dev = 0;
    CSD_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return CSD_ERR_UNSUPPORTED;
    char* ws = nullptr;
    {
        std::lock_guard<std::mutex> lk(g_accept_scratch_mu);
        if (!g_accept_scratch_ptr[dev]) {
            void* p = nullptr;
            CSD_CUDA(cudaGetSymbolAddress(&p, g_accept_scratch));
            g_accept_scratch_ptr[dev] = p;
        }
        ws = (char*)g_accept_scratch_ptr[dev];
    }
    // (bad token ids are not recorded in the status word here: looking that word up may allocate)
    return run_accept(target_logits_dev, draft_logits_dev, onehot_dev, draft_tokens_dev, rows, k, V, temperature, lenience,
                      seed, step, n_accepted_dev, out_token_dev, ws, L, nullptr, (cudaStream_t)stream);
}
