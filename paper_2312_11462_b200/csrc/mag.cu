// Max-Gram statistical drafter (Section 3.3, Appendix A) on a hashed n-gram table.
//
// Build: every n-gram of the haystack of order 1..max_order that is followed by at least one
// haystack token is inserted into one open-addressing table.  A slot holds (start << 6 | order)
// of the EARLIEST occurrence of its n-gram; slot identity is decided by comparing haystack
// tokens, never by the hash alone, so collisions cannot change the result.
// Draft: one warp; lane o-1 probes the table for the suffix of order o, the longest hit wins
// (a suffix of order o that matches implies every shorter one matches), then the tokens after
// the hit are copied; without a hit one token comes from the bigram table.
//
// Dynamic haystack (Section 3.3 lets the match come from the input or from the existing
// generation): the haystack is the static one followed by the generated part of the sequence,
// seq[gen_from, T).  The table still covers every occurrence that ends at least two tokens before
// the end of the static part; occurrences that end later (their follower, or part of them, is
// generated text, which comes and goes as blocks are rejected) are few and are found by a direct
// scan: every lane takes candidate end positions in turn, counts how far the text before them
// agrees with the sequence's tail, and records the earliest end per order.  Table hits start
// earlier than scanned ones by construction, so per order the table wins when it has a hit.
#include "common.cuh"

struct csd_mag {
    const int32_t* hay;
    const int32_t* bigram;
    int L, V, max_order, slots;
    int* table;
};

namespace csd {

constexpr int EMPTY_SLOT = 0x7fffffff;

__device__ __forceinline__ uint32_t gram_hash(const int32_t* g, int order) {
    uint32_t h = 0x811C9DC5u ^ (uint32_t)order * 0x9E3779B1u;
    for (int i = 0; i < order; ++i) {
        h ^= (uint32_t)g[i];
        h *= 0x01000193u;
        h ^= h >> 15;
    }
    h ^= h >> 13; h *= 0x5bd1e995u; h ^= h >> 16;
    return h;
}

__device__ __forceinline__ bool same_gram(const int32_t* a, const int32_t* b, int order) {
    for (int i = 0; i < order; ++i)
        if (a[i] != b[i]) return false;
    return true;
}

__global__ void mag_fill_kernel(int* table, int slots) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < slots) table[i] = EMPTY_SLOT;
}

__global__ void mag_build_kernel(const int32_t* __restrict__ hay, int L, int max_order, int* table, int slots,
                                 int* status) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    const int j = idx / max_order, order = idx % max_order + 1;
    if (j >= L || j + order > L - 1) return;   // needs a following token inside the haystack
    const int mine = (j << 6) | order;
    uint32_t h = gram_hash(hay + j, order) & (uint32_t)(slots - 1);
    for (int probe = 0; probe < slots; ++probe) {
        int cur = table[h];
        if (cur == EMPTY_SLOT) {
            int prev = atomicCAS(&table[h], EMPTY_SLOT, mine);
            if (prev == EMPTY_SLOT) return;
            cur = prev;
        }
        // a claimed slot only ever changes to an earlier start of the same n-gram
        if ((cur & 63) == order && same_gram(hay + (cur >> 6), hay + j, order)) {
            atomicMin(&table[h], mine);
            return;
        }
        h = (h + 1) & (uint32_t)(slots - 1);
    }
    set_status(status, CSD_ERR_TIMEOUT);       // table full: cannot happen with slots >= n-grams
}

constexpr int MAG_MAX_N = 64;

__global__ void __launch_bounds__(32)
mag_draft_kernel(const int32_t* __restrict__ hay, int L, const int32_t* __restrict__ bigram, int V,
                 const int* __restrict__ table, int slots, int max_order, const int32_t* seq, int T,
                 int gen_from, int n, int32_t* out, int* status) {
    // joined haystack: hay[0, L) followed by seq[gen_from, T) when gen_from >= 0
    const int G = gen_from >= 0 ? T - gen_from : 0, LJ = L + G;
    auto joined = [&](int i) { return i < L ? hay[i] : seq[gen_from + (i - L)]; };
    __shared__ int best_end[CSD_MAG_MAX_ORDER + 1];
    // tail = last max_order tokens of the sequence followed by the tokens proposed so far
    // (at most CSD_MAG_MAX_ORDER + MAG_MAX_N entries, so it never overflows)
    __shared__ int32_t tail[CSD_MAG_MAX_ORDER + MAG_MAX_N];
    const int lane = threadIdx.x;
    const int keep = T < max_order ? T : max_order;
    for (int i = lane; i < keep; i += 32) tail[i] = seq[T - keep + i];
    __syncwarp();
    int len = keep;       // valid tokens in tail
    int total = T;        // length of the (virtual) full sequence
    int made = 0;
    while (made < n) {
        const int limit = min(min(total, max_order), len);
        const int order = lane + 1;
        int hit = -1;
        if (order <= limit && slots > 0) {
            const int32_t* g = tail + len - order;
            uint32_t h = gram_hash(g, order) & (uint32_t)(slots - 1);
            for (int probe = 0; probe < slots; ++probe) {
                int cur = table[h];
                if (cur == EMPTY_SLOT) break;
                if ((cur & 63) == order && same_gram(hay + (cur >> 6), g, order)) { hit = cur >> 6; break; }
                h = (h + 1) & (uint32_t)(slots - 1);
            }
        }
        if (G > 0) {
            // ends e in [L-1, LJ-2]: the occurrence's follower e+1 exists and is generated text
            best_end[lane + 1] = 0x7fffffff;
            __syncwarp();
            for (int e = max(L - 1, 0) + lane; e <= LJ - 2; e += 32) {
                int agree = 0;
                while (agree < limit && agree <= e && joined(e - agree) == tail[len - 1 - agree]) ++agree;
                for (int o = 1; o <= agree; ++o) atomicMin(&best_end[o], e);
            }
            __syncwarp();
            if (hit < 0 && order <= limit && best_end[order] != 0x7fffffff) hit = best_end[order] - order + 1;
            __syncwarp();
        }
        const unsigned ballot = __ballot_sync(0xffffffffu, hit >= 0);
        if (ballot == 0) {
            int32_t last = tail[len - 1];
            int32_t nx = 0;
            if (last >= 0 && last < V) nx = bigram[last];
            else if (lane == 0) set_status(status, CSD_ERR_BAD_TOKEN);
            if (lane == 0) { tail[len] = nx; out[made] = nx; }
            len += 1; total += 1; made += 1;
        } else {
            const int best = 31 - __clz(ballot);              // lane of the longest order that hit
            const int start = __shfl_sync(0xffffffffu, hit, best);
            int idx = start + best + 1;                      // haystack index of the next token
            int cnt = min(n - made, LJ - idx);
            for (int i = lane; i < cnt; i += 32) {
                int32_t t = joined(idx + i);
                tail[len + i] = t;
                out[made + i] = t;
            }
            len += cnt; total += cnt; made += cnt;
        }
        __syncwarp();
    }
}

static int default_slots(int L, int max_order) {
    long long grams = (long long)L * max_order * 2;
    int s = 64;
    while (s < grams) s <<= 1;
    return s;
}

}  // namespace csd

using namespace csd;

extern "C" size_t csd_mag_workspace_bytes(int L, int max_order, int table_slots) {
    if (L < 0 || max_order < 1 || max_order > CSD_MAG_MAX_ORDER) return 0;
    int slots = table_slots > 0 ? table_slots : default_slots(L, max_order);
    return align_up((size_t)slots * sizeof(int), 256);
}

extern "C" csd_status csd_mag_create(const int32_t* haystack_dev, int L, int V, const int32_t* bigram_next_dev,
                                     int max_order, int table_slots, void* workspace_dev, size_t workspace_bytes,
                                     void* stream, csd_mag** out) {
    if (!out) return CSD_ERR_INVALID_ARG;
    *out = nullptr;
    if (L < 0 || V < 1 || !bigram_next_dev || (L > 0 && !haystack_dev) || !workspace_dev) return CSD_ERR_INVALID_ARG;
    if (max_order < 1 || max_order > CSD_MAG_MAX_ORDER) return CSD_ERR_INVALID_ARG;
    if (L >= (1 << 24)) return CSD_ERR_CAPACITY;
    int slots = table_slots > 0 ? table_slots : default_slots(L, max_order);
    if (slots & (slots - 1)) return CSD_ERR_INVALID_ARG;
    // n-grams that get inserted: orders 1..max_order with a following token
    long long grams = 0;
    for (int o = 1; o <= max_order; ++o) grams += L - o > 0 ? L - o : 0;
    if (slots < grams + 1) return CSD_ERR_CAPACITY;
    if (workspace_bytes < (size_t)slots * sizeof(int)) return CSD_ERR_CAPACITY;
    int* status = status_word_device();
    if (!status) return CSD_ERR_CUDA;
    csd_mag* g = (csd_mag*)malloc(sizeof(csd_mag));
    if (!g) return CSD_ERR_OOM;
    g->hay = haystack_dev; g->bigram = bigram_next_dev; g->L = L; g->V = V; g->max_order = max_order;
    g->slots = slots; g->table = (int*)workspace_dev;
    cudaStream_t st = (cudaStream_t)stream;
    mag_fill_kernel<<<(slots + 255) / 256, 256, 0, st>>>(g->table, slots);
    count_launch();
    long long work = (long long)L * max_order;
    if (work > 0) {
        mag_build_kernel<<<(unsigned)((work + 127) / 128), 128, 0, st>>>(haystack_dev, L, max_order, g->table, slots, status);
        count_launch();
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { free(g); return note_cuda(e); }
    *out = g;
    return CSD_OK;
}

extern "C" csd_status csd_mag_destroy(csd_mag* g) {
    free(g);
    return CSD_OK;
}

static csd_status mag_draft(csd_mag* g, const int32_t* seq_dev, int T, int gen_from, int n, int32_t* out_tokens_dev,
                            void* stream) {
    if (!g || !seq_dev || !out_tokens_dev || T < 1) return CSD_ERR_INVALID_ARG;
    if (n < 1 || n > MAG_MAX_N) return CSD_ERR_INVALID_ARG;
    int* status = status_word_device();
    if (!status) return CSD_ERR_CUDA;
    mag_draft_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(g->hay, g->L, g->bigram, g->V, g->table, g->slots,
                                                          g->max_order, seq_dev, T, gen_from, n, out_tokens_dev, status);
    count_launch();
    CSD_CUDA(cudaGetLastError());
    return CSD_OK;
}

extern "C" csd_status csd_mag_draft(csd_mag* g, const int32_t* seq_dev, int T, int n, int32_t* out_tokens_dev,
                                    void* stream) {
    return mag_draft(g, seq_dev, T, -1, n, out_tokens_dev, stream);
}

extern "C" csd_status csd_mag_draft_dynamic(csd_mag* g, const int32_t* seq_dev, int T, int gen_from, int n,
                                            int32_t* out_tokens_dev, void* stream) {
    if (gen_from < 0 || gen_from > T) return CSD_ERR_INVALID_ARG;
    return mag_draft(g, seq_dev, T, gen_from, n, out_tokens_dev, stream);
}
