// Review rule of speculative sampling (Section 2; lenience / greedy: Section 3.1) as three
// passes over the vocabulary:
//   stats   one streaming pass over all (2k+1) logit vectors of every row: per-chunk max,
//           arg-max and sum of exponentials (fp32).  This is the HBM-bound part.
//   decide  per row: merge the chunk partials, run the accept tests left to right with the
//           Philox uniforms, find the first rejection n.
//   resample (temperature > 0 only) per row, at position n only: total mass of the residual
//           max(0, p - q) (or of p after k acceptances) and the inverse-CDF pick, in fp64 so
//           that the chosen token does not depend on the summation order.
#include "common.cuh"
#include "philox.cuh"
#include <mutex>

namespace csd {

constexpr int ST_THREADS = 256;
constexpr int ST_CHUNK = 4096;   // logits per CTA of the stats pass
constexpr int RS_THREADS = 256;
constexpr int RS_PER_THREAD = 8;
constexpr int RS_CHUNK = RS_THREADS * RS_PER_THREAD;  // logits per CTA of the resample passes

struct __align__(16) StatPartial {
    float mx;
    float sum;   // sum exp((x - mx) * invT) over the chunk
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
// stats pass
// ---------------------------------------------------------------------------------------------
template <bool VEC>
__global__ void __launch_bounds__(ST_THREADS)
accept_stats_kernel(const float* __restrict__ tl, const float* __restrict__ dl, long long n_tvec, int V,
                    float invT, int greedy, StatPartial* __restrict__ out, int nchunk) {
    const long long vec = blockIdx.x;
    const int chunk = blockIdx.y;
    const float* src = vec < n_tvec ? tl + vec * (long long)V : dl + (vec - n_tvec) * (long long)V;
    const int base = chunk * ST_CHUNK;
    const int tid = threadIdx.x;
    constexpr int PER = ST_CHUNK / ST_THREADS;  // 16
    float v[PER];
    if (VEC) {
#pragma unroll
        for (int j = 0; j < PER / 4; ++j) {
            int e = base + 4 * (tid + ST_THREADS * j);
            float4 f = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
            if (e < V) f = __ldcs(reinterpret_cast<const float4*>(src + e));
            v[4 * j + 0] = f.x; v[4 * j + 1] = f.y; v[4 * j + 2] = f.z; v[4 * j + 3] = f.w;
        }
    } else {
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            int e = base + tid + ST_THREADS * j;
            v[j] = e < V ? __ldcs(src + e) : -INFINITY;
        }
    }
    // thread-local max with the smallest index attaining it
    float mx = -INFINITY;
    int arg = 0x7fffffff;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        int e = VEC ? base + 4 * (tid + ST_THREADS * (j / 4)) + (j & 3) : base + tid + ST_THREADS * j;
        if (v[j] > mx || (v[j] == mx && e < arg)) { mx = v[j]; arg = e; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        float om = __shfl_xor_sync(0xffffffffu, mx, o);
        int oa = __shfl_xor_sync(0xffffffffu, arg, o);
        if (om > mx || (om == mx && oa < arg)) { mx = om; arg = oa; }
    }
    __shared__ float s_mx[ST_THREADS / 32];
    __shared__ int s_arg[ST_THREADS / 32];
    __shared__ float s_sum[ST_THREADS / 32];
    const int warp = tid >> 5, lane = tid & 31;
    if (lane == 0) { s_mx[warp] = mx; s_arg[warp] = arg; }
    __syncthreads();
    mx = s_mx[0]; arg = s_arg[0];
#pragma unroll
    for (int w = 1; w < ST_THREADS / 32; ++w)
        if (s_mx[w] > mx || (s_mx[w] == mx && s_arg[w] < arg)) { mx = s_mx[w]; arg = s_arg[w]; }
    float sum = 0.f;
    if (!greedy && mx > -INFINITY) {
#pragma unroll
        for (int j = 0; j < PER; ++j) sum += __expf((v[j] - mx) * invT);
    }
    sum = warp_sum(sum);
    if (lane == 0) s_sum[warp] = sum;
    __syncthreads();
    if (tid == 0) {
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < ST_THREADS / 32; ++w) tot += s_sum[w];
        StatPartial p;
        p.mx = mx; p.sum = tot; p.arg = arg; p.pad = 0;
        out[vec * nchunk + chunk] = p;
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
                     int* __restrict__ n_acc, int* __restrict__ out_tok, RowInfo* __restrict__ info, int* status) {
    const int row = blockIdx.x;
    __shared__ float s_mx[2 * MAX_K + 1];
    __shared__ float s_z[2 * MAX_K + 1];
    __shared__ int s_arg[2 * MAX_K + 1];
    const bool greedy = temperature == 0.f;
    const float invT = greedy ? 1.f : 1.f / temperature;
    const int nvec_row = dl ? 2 * k + 1 : k + 1;
    const long long n_tvec = (long long)rows * (k + 1);
    for (int i = threadIdx.x; i < nvec_row; i += blockDim.x) {
        long long vec = i <= k ? (long long)row * (k + 1) + i : n_tvec + (long long)row * k + (i - k - 1);
        const StatPartial* p = part + vec * nchunk;
        float mx = p[0].mx;
        int arg = p[0].arg;
        for (int c = 1; c < nchunk; ++c)
            if (p[c].mx > mx) { mx = p[c].mx; arg = p[c].arg; }
        float z = 0.f;
        if (!greedy)
            for (int c = 0; c < nchunk; ++c)
                if (p[c].mx > -INFINITY) z += p[c].sum * __expf((p[c].mx - mx) * invT);
        s_mx[i] = mx; s_z[i] = z; s_arg[i] = arg;
    }
    __syncthreads();
    if (threadIdx.x != 0) return;
    const int* tok = tokens + (long long)row * k;
    RowInfo ri;
    ri.n = k; ri.mode = MODE_DONE; ri.x = 0; ri.pad = 0; ri.max_t = 0; ri.max_q = 0; ri.u2 = 0;
    if (greedy) {
        int n = 0;
        while (n < k && tok[n] == s_arg[n]) ++n;
        n_acc[row] = n;
        out_tok[row] = s_arg[n];
        ri.n = n;
        info[row] = ri;
        return;
    }
    const uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
    const uint32_t c2 = (uint32_t)step, c3 = (uint32_t)(step >> 32);
    const double T = (double)temperature;
    int n = k;
    for (int i = 0; i < k; ++i) {
        int x = tok[i];
        Philox4 r = philox4x32_10((uint32_t)i, (uint32_t)row, c2, c3, k0, k1);
        const bool point = dl == nullptr || (onehot && onehot[(long long)row * k + i] != 0);
        bool accept = false;
        if (x < 0 || x >= V) {
            set_status(status, CSD_ERR_BAD_TOKEN);
            x = 0;
        } else {
            double u = word_uniform(r.w[0]);
            double px = exp(((double)tl[((long long)row * (k + 1) + i) * V + x] - (double)s_mx[i]) / T) / (double)s_z[i];
            double qx = 1.0;
            if (!point)
                qx = exp(((double)dl[((long long)row * k + i) * V + x] - (double)s_mx[k + 1 + i]) / T) /
                     (double)s_z[k + 1 + i];
            accept = u * qx < (double)lenience * px;
        }
        if (!accept) {
            n = i;
            ri.mode = point ? MODE_RESID_POINT : MODE_RESID_LOGITS;
            ri.x = x;
            ri.max_t = (double)s_mx[i];
            ri.max_q = point ? 0.0 : (double)s_mx[k + 1 + i];
            ri.u2 = word_uniform(r.w[1]);
            break;
        }
    }
    if (n == k) {
        Philox4 r = philox4x32_10((uint32_t)k, (uint32_t)row, c2, c3, k0, k1);
        ri.mode = MODE_TARGET_ONLY;
        ri.max_t = (double)s_mx[k];
        ri.u2 = word_uniform(r.w[1]);
    }
    ri.n = n;
    n_acc[row] = n;
    info[row] = ri;
}

// ---------------------------------------------------------------------------------------------
// resample passes (fp64).  grid = (rows, chunks)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ double block_sum_ordered(double v, double* s_warp) {
    // fixed reduction tree: lanes by xor-shuffle, then warps in index order
    v = warp_sum(v);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) s_warp[warp] = v;
    __syncthreads();
    double tot = 0.0;
    for (int w = 0; w < RS_THREADS / 32; ++w) tot += s_warp[w];
    return tot;
}

// pass 1: per-chunk sums of exp((t - max_t)/T) and exp((d - max_q)/T)
__global__ void __launch_bounds__(RS_THREADS)
resample_z_kernel(const float* __restrict__ tl, const float* __restrict__ dl, int k, int V, float temperature,
                  const RowInfo* __restrict__ info, double2* __restrict__ zpart, int nchunk) {
    const int row = blockIdx.x, chunk = blockIdx.y;
    const RowInfo ri = info[row];
    if (ri.mode == MODE_DONE) return;
    __shared__ double s_warp[RS_THREADS / 32];
    const double T = (double)temperature;
    const float* t = tl + ((long long)row * (k + 1) + ri.n) * V;
    const float* d = ri.mode == MODE_RESID_LOGITS ? dl + ((long long)row * k + ri.n) * V : nullptr;
    const int e0 = chunk * RS_CHUNK + threadIdx.x * RS_PER_THREAD;
    double sp = 0.0, sq = 0.0;
#pragma unroll
    for (int j = 0; j < RS_PER_THREAD; ++j) {
        int e = e0 + j;
        if (e < V) {
            sp += exp(((double)t[e] - ri.max_t) / T);
            if (d) sq += exp(((double)d[e] - ri.max_q) / T);
        }
    }
    sp = block_sum_ordered(sp, s_warp);
    sq = block_sum_ordered(sq, s_warp);
    if (threadIdx.x == 0) zpart[(long long)row * nchunk + chunk] = make_double2(sp, sq);
}

__device__ __forceinline__ double residual_value(double ep, double eq, double Zp, double Zq, int mode, int e, int x) {
    double p = ep / Zp;
    if (mode == MODE_TARGET_ONLY) return p;
    double q = mode == MODE_RESID_POINT ? (e == x ? 1.0 : 0.0) : eq / Zq;
    double r = p - q;
    return r > 0.0 ? r : 0.0;
}

// pass 2: per-chunk mass of the residual
__global__ void __launch_bounds__(RS_THREADS)
resample_mass_kernel(const float* __restrict__ tl, const float* __restrict__ dl, int k, int V, float temperature,
                     const RowInfo* __restrict__ info, const double2* __restrict__ zpart,
                     double* __restrict__ rpart, int nchunk) {
    const int row = blockIdx.x, chunk = blockIdx.y;
    const RowInfo ri = info[row];
    if (ri.mode == MODE_DONE) return;
    __shared__ double s_warp[RS_THREADS / 32];
    __shared__ double s_Z[2];
    if (threadIdx.x == 0) {
        double Zp = 0.0, Zq = 0.0;
        for (int c = 0; c < nchunk; ++c) {
            double2 z = zpart[(long long)row * nchunk + c];
            Zp += z.x; Zq += z.y;
        }
        s_Z[0] = Zp; s_Z[1] = Zq;
    }
    __syncthreads();
    const double Zp = s_Z[0], Zq = s_Z[1], T = (double)temperature;
    const float* t = tl + ((long long)row * (k + 1) + ri.n) * V;
    const float* d = ri.mode == MODE_RESID_LOGITS ? dl + ((long long)row * k + ri.n) * V : nullptr;
    const int e0 = chunk * RS_CHUNK + threadIdx.x * RS_PER_THREAD;
    double s = 0.0;
#pragma unroll
    for (int j = 0; j < RS_PER_THREAD; ++j) {
        int e = e0 + j;
        if (e < V) {
            double ep = exp(((double)t[e] - ri.max_t) / T);
            double eq = d ? exp(((double)d[e] - ri.max_q) / T) : 0.0;
            s += residual_value(ep, eq, Zp, Zq, ri.mode, e, ri.x);
        }
    }
    s = block_sum_ordered(s, s_warp);
    if (threadIdx.x == 0) rpart[(long long)row * nchunk + chunk] = s;
}

// pass 3: one CTA per row picks the token
__global__ void __launch_bounds__(RS_THREADS)
resample_pick_kernel(const float* __restrict__ tl, const float* __restrict__ dl, int k, int V, float temperature,
                     const RowInfo* __restrict__ info, const double2* __restrict__ zpart,
                     const double* __restrict__ rpart, int nchunk, int* __restrict__ out_tok) {
    const int row = blockIdx.x;
    const RowInfo ri = info[row];
    if (ri.mode == MODE_DONE) return;
    __shared__ double s_d[4];   // Zp, Zq, target, base
    __shared__ int s_i[3];      // chunk, mode, forced-last flag
    __shared__ double s_scan[RS_THREADS / 32];
    __shared__ int s_pick, s_last;
    if (threadIdx.x == 0) {
        double Zp = 0.0, Zq = 0.0, S = 0.0;
        for (int c = 0; c < nchunk; ++c) {
            double2 z = zpart[(long long)row * nchunk + c];
            Zp += z.x; Zq += z.y;
            S += rpart[(long long)row * nchunk + c];
        }
        int mode = ri.mode;
        const bool empty = !(S > 0.0) || !isfinite(S);
        if (empty) {   // empty residual: fall back to the target law itself
            mode = MODE_TARGET_ONLY;
            S = 0.0;
            for (int c = 0; c < nchunk; ++c) S += zpart[(long long)row * nchunk + c].x / Zp;
        }
        const double target = ri.u2 * S;
        double cum = 0.0, base = 0.0;
        int chunk = -1, last_pos = 0;
        for (int c = 0; c < nchunk; ++c) {
            double mass = empty ? zpart[(long long)row * nchunk + c].x / Zp : rpart[(long long)row * nchunk + c];
            if (mass > 0.0) last_pos = c;
            if (cum + mass > target) { chunk = c; base = cum; break; }
            cum += mass;
        }
        int forced = 0;
        if (chunk < 0) { chunk = last_pos; forced = 1; }
        s_d[0] = Zp; s_d[1] = Zq; s_d[2] = target; s_d[3] = base;
        s_i[0] = chunk; s_i[1] = mode; s_i[2] = forced;
        s_pick = 0x7fffffff; s_last = -1;
    }
    __syncthreads();
    const double Zp = s_d[0], Zq = s_d[1], target = s_d[2], base = s_d[3], T = (double)temperature;
    const int chunk = s_i[0], mode = s_i[1], forced = s_i[2];
    const float* t = tl + ((long long)row * (k + 1) + ri.n) * V;
    const float* d = mode == MODE_RESID_LOGITS ? dl + ((long long)row * k + ri.n) * V : nullptr;
    const int e0 = chunk * RS_CHUNK + threadIdx.x * RS_PER_THREAD;
    double r[RS_PER_THREAD];
    double local = 0.0;
    int my_last = -1;
#pragma unroll
    for (int j = 0; j < RS_PER_THREAD; ++j) {
        int e = e0 + j;
        r[j] = 0.0;
        if (e < V) {
            double ep = exp(((double)t[e] - ri.max_t) / T);
            double eq = d ? exp(((double)d[e] - ri.max_q) / T) : 0.0;
            r[j] = residual_value(ep, eq, Zp, Zq, mode, e, ri.x);
            if (r[j] > 0.0) my_last = e;
        }
        local += r[j];
    }
    // exclusive prefix of the per-thread sums, in thread order
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    double incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        double up = __shfl_up_sync(0xffffffffu, incl, o);
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
    if (threadIdx.x == 0) {
        int pick = s_pick != 0x7fffffff ? s_pick : (s_last >= 0 ? s_last : 0);
        out_tok[row] = pick;
    }
}

struct AcceptLayout {
    size_t part_off, info_off, z_off, r_off, total;
    int nchunk_a, nchunk_r;
};

static AcceptLayout accept_layout(int rows, int k, int V) {
    AcceptLayout L;
    L.nchunk_a = (V + ST_CHUNK - 1) / ST_CHUNK;
    L.nchunk_r = (V + RS_CHUNK - 1) / RS_CHUNK;
    size_t nvec = (size_t)rows * (2 * (size_t)k + 1);
    size_t off = 0;
    L.part_off = off; off = align_up(off + nvec * L.nchunk_a * sizeof(StatPartial), 256);
    L.info_off = off; off = align_up(off + (size_t)rows * sizeof(RowInfo), 256);
    L.z_off = off;    off = align_up(off + (size_t)rows * L.nchunk_r * sizeof(double2), 256);
    L.r_off = off;    off = align_up(off + (size_t)rows * L.nchunk_r * sizeof(double), 256);
    L.total = off;
    return L;
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
    if (L.nchunk_a > 65535 || L.nchunk_r > 65535) return CSD_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    int* status = status_word_device();
    if (!status) return CSD_ERR_CUDA;
    char* ws = (char*)workspace_dev;
    StatPartial* part = (StatPartial*)(ws + L.part_off);
    RowInfo* info = (RowInfo*)(ws + L.info_off);
    double2* zpart = (double2*)(ws + L.z_off);
    double* rpart = (double*)(ws + L.r_off);
    const bool greedy = temperature == 0.f;
    const float invT = greedy ? 1.f : 1.f / temperature;
    const bool use_d = draft_logits_dev != nullptr && k > 0 && !greedy;
    const float* dl = use_d ? draft_logits_dev : nullptr;
    const long long n_tvec = (long long)rows * (k + 1);
    const long long nvec = n_tvec + (use_d ? (long long)rows * k : 0);
    if (nvec > 0x7fffffffLL) return CSD_ERR_UNSUPPORTED;
    const bool vec_ok = (V % 4 == 0) && (((uintptr_t)target_logits_dev & 15) == 0) &&
                        (!use_d || ((uintptr_t)draft_logits_dev & 15) == 0);
    dim3 grid((unsigned)nvec, (unsigned)L.nchunk_a);
    if (vec_ok)
        accept_stats_kernel<true><<<grid, ST_THREADS, 0, st>>>(target_logits_dev, dl, n_tvec, V, invT, greedy, part, L.nchunk_a);
    else
        accept_stats_kernel<false><<<grid, ST_THREADS, 0, st>>>(target_logits_dev, dl, n_tvec, V, invT, greedy, part, L.nchunk_a);
    accept_decide_kernel<<<rows, 128, 0, st>>>(target_logits_dev, dl, onehot_dev, draft_tokens_dev, rows, k, V,
                                               temperature, lenience, seed, step, part, L.nchunk_a,
                                               n_accepted_dev, out_token_dev, info, status);
    count_launch(2);
    if (!greedy) {
        dim3 g2((unsigned)rows, (unsigned)L.nchunk_r);
        resample_z_kernel<<<g2, RS_THREADS, 0, st>>>(target_logits_dev, dl, k, V, temperature, info, zpart, L.nchunk_r);
        resample_mass_kernel<<<g2, RS_THREADS, 0, st>>>(target_logits_dev, dl, k, V, temperature, info, zpart, rpart, L.nchunk_r);
        resample_pick_kernel<<<rows, RS_THREADS, 0, st>>>(target_logits_dev, dl, k, V, temperature, info, zpart, rpart,
                                                          L.nchunk_r, out_token_dev);
        count_launch(3);
    }
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
    if (L.nchunk_a > 65535 || L.nchunk_r > 65535) return CSD_ERR_UNSUPPORTED;
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
    cudaStream_t st = (cudaStream_t)stream;
    StatPartial* part = (StatPartial*)(ws + L.part_off);
    RowInfo* info = (RowInfo*)(ws + L.info_off);
    double2* zpart = (double2*)(ws + L.z_off);
    double* rpart = (double*)(ws + L.r_off);
    const bool greedy = temperature == 0.f;
    const float invT = greedy ? 1.f : 1.f / temperature;
    const bool use_d = draft_logits_dev != nullptr && k > 0 && !greedy;
    const float* dl = use_d ? draft_logits_dev : nullptr;
    const long long n_tvec = (long long)rows * (k + 1);
    const long long nvec = n_tvec + (use_d ? (long long)rows * k : 0);
    if (nvec > 0x7fffffffLL) return CSD_ERR_UNSUPPORTED;
    const bool vec_ok = (V % 4 == 0) && (((uintptr_t)target_logits_dev & 15) == 0) &&
                        (!use_d || ((uintptr_t)draft_logits_dev & 15) == 0);
    // Every word of the scratch that a pass reads is written by an earlier pass of the same call,
    // so nothing has to be cleared even though the array still holds the previous call's data.
    dim3 grid((unsigned)nvec, (unsigned)L.nchunk_a);
    if (vec_ok)
        accept_stats_kernel<true><<<grid, ST_THREADS, 0, st>>>(target_logits_dev, dl, n_tvec, V, invT, greedy, part, L.nchunk_a);
    else
        accept_stats_kernel<false><<<grid, ST_THREADS, 0, st>>>(target_logits_dev, dl, n_tvec, V, invT, greedy, part, L.nchunk_a);
    accept_decide_kernel<<<rows, 128, 0, st>>>(target_logits_dev, dl, onehot_dev, draft_tokens_dev, rows, k, V,
                                               temperature, lenience, seed, step, part, L.nchunk_a,
                                               n_accepted_dev, out_token_dev, info, nullptr);
    count_launch(2);
    if (!greedy) {
        dim3 g2((unsigned)rows, (unsigned)L.nchunk_r);
        resample_z_kernel<<<g2, RS_THREADS, 0, st>>>(target_logits_dev, dl, k, V, temperature, info, zpart, L.nchunk_r);
        resample_mass_kernel<<<g2, RS_THREADS, 0, st>>>(target_logits_dev, dl, k, V, temperature, info, zpart, rpart, L.nchunk_r);
        resample_pick_kernel<<<rows, RS_THREADS, 0, st>>>(target_logits_dev, dl, k, V, temperature, info, zpart, rpart,
                                                          L.nchunk_r, out_token_dev);
        count_launch(3);
    }
    CSD_CUDA(cudaGetLastError());
    return CSD_OK;
}
