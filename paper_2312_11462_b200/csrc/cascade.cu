// Algorithm 1 (CascadeSpeculativeDraftingStep) as a host driver over the device kernels: the
// for-loop over slots is the horizontal cascade, the recursion the vertical cascade, Max-Gram
// the base case.  Tokens, logits and laws stay on the device; per review the host reads back
// two integers (accepted count, output token).
#include <chrono>
#include <mutex>
#include <string.h>
#include <vector>
#include "model.cuh"

namespace csd {

constexpr int RING = 128;   // proposing laws are kept for the last RING positions

struct CascadeWs {
    size_t seq, hay, mag, law, qlaw, dl, onehot, result, accept, total;
};

static CascadeWs cascade_layout(int V, int max_block, int cap, int L, int max_order) {
    CascadeWs w{};
    size_t off = 0;
    auto put = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    w.seq = put(((size_t)cap + 64) * 4);
    w.hay = put((size_t)(L > 0 ? L : 1) * 4);
    w.mag = put(csd_mag_workspace_bytes(L, max_order, 0));
    w.law = put((size_t)CSD_MAX_ROWS * V * 4);            // a forward may carry up to CSD_MAX_ROWS rows (catch-up chunks)
    w.qlaw = put((size_t)RING * V * 4);
    w.dl = put((size_t)(max_block > 0 ? max_block : 1) * V * 4);
    w.onehot = put((size_t)(max_block + 1) * 4);
    w.result = put(64);
    w.accept = put(csd_spec_accept_workspace_bytes(1, max_block, V));
    w.total = off;
    return w;
}

// Host-side resources of a generation (a small block of mapped pinned memory for the results of
// the accept kernels, three events): created once per device and kept, so that a call creates and
// frees nothing; a second call that overlaps the first on the same device makes its own.
struct HostKit {
    int32_t* pinned = nullptr; int32_t* mapped = nullptr; cudaEvent_t ev[3] = {nullptr, nullptr, nullptr};
    bool pooled = false;
};
constexpr int KIT_WORDS = 2 + CSD_MAX_ROWS + 64, KIT_DEVICES = 64;
static std::mutex g_kit_mu;
static HostKit g_kit[KIT_DEVICES];
static bool g_kit_busy[KIT_DEVICES];

static void kit_free(HostKit& k) {
    for (cudaEvent_t& e : k.ev) { if (e) cudaEventDestroy(e); e = nullptr; }
    if (k.pinned) cudaFreeHost(k.pinned);
    k.pinned = nullptr; k.mapped = nullptr;
}
static csd_status kit_make(HostKit& k) {
    if (cudaHostAlloc((void**)&k.pinned, (size_t)KIT_WORDS * 4, cudaHostAllocMapped) != cudaSuccess ||
        cudaHostGetDevicePointer((void**)&k.mapped, k.pinned, 0) != cudaSuccess || !k.mapped) {
        const csd_status s = note_cuda(cudaGetLastError());
        kit_free(k);
        return s != CSD_OK ? s : CSD_ERR_CUDA;
    }
    for (cudaEvent_t& e : k.ev)
        if (cudaEventCreate(&e) != cudaSuccess) { const csd_status s = note_cuda(cudaGetLastError()); kit_free(k); return s; }
    return CSD_OK;
}
static csd_status kit_acquire(HostKit& out) {
    int dev = 0;
    CSD_CUDA(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lk(g_kit_mu);
    if (dev >= 0 && dev < KIT_DEVICES && !g_kit_busy[dev]) {
        if (!g_kit[dev].pinned) {
            const csd_status s = kit_make(g_kit[dev]);
            if (s != CSD_OK) return s;
        }
        g_kit_busy[dev] = true;
        out = g_kit[dev];
        out.pooled = true;
        return CSD_OK;
    }
    out = HostKit{};
    return kit_make(out);
}
static void kit_release(HostKit& k) {
    if (!k.pinned) return;
    if (k.pooled) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) dev = -1;
        std::lock_guard<std::mutex> lk(g_kit_mu);
        for (int d = 0; d < KIT_DEVICES; ++d)
            if (g_kit[d].pinned == k.pinned) g_kit_busy[d] = false;
    } else {
        kit_free(k);
    }
    k.pinned = nullptr;
}

struct Gen {
    csd_model* const* models; int n_levels; const int32_t* K; int max_block; float lenience, temperature;
    uint64_t seed, step = 0; csd_mag* mag = nullptr; int V, cap; int dynamic = 0, init_len = 0;
    int32_t* seq; int len = 0; int kv[8] = {0};
    std::vector<signed char> src;        // per position: proposing level, -1 = point mass
    float *law, *qlaw, *dl; int32_t *onehot_dev, *result_dev, *result_map = nullptr; void* accept_ws; size_t accept_bytes;
    int32_t* pinned = nullptr;           // [0..1] = (n_acc, out_tok); [2..] = onehot flags staging
    csd_cascade_stats* st; cudaStream_t stream;
    cudaEvent_t ev_decode; bool decode_marked = false;
};

// forward `cnt` rows of level r starting at sequence position `from`; logits land in g.law, or
// nowhere when nobody reads them (prompt prefill, catch-up chunks before the reviewed block)
static csd_status forward(Gen& g, int r, int from, int cnt, bool want_logits = true) {
    csd_status s = csd_review_forward(g.models[r], g.seq + from, cnt, from, want_logits ? g.law : nullptr, g.stream);
    g.st->forwards[r] += 1;
    return s;
}

static csd_status step(Gen& g, int r, int budget);

static csd_status review(Gen& g, int r, int P, int nd) {
    // a forward carries as many rows as the model takes: fewer passes over the weights while catching up
    const int V = g.V, maxrows = g.models[r]->cfg.max_rows < CSD_MAX_ROWS ? g.models[r]->cfg.max_rows : CSD_MAX_ROWS;
    int from = g.kv[r] < P - 1 ? g.kv[r] : P - 1;
    int cnt = 0;
    while (from < P + nd) {   // catch up on tokens this level has not cached, then the block itself
        cnt = P + nd - from;
        if (cnt > maxrows) cnt = (from + maxrows <= P - 1) ? maxrows : (P - 1) - from;
        CSD_CUDA(cudaGetLastError());
        csd_status s = forward(g, r, from, cnt, from + cnt == P + nd);
        if (s != CSD_OK) return s;
        from += cnt;
    }
    const float* target = g.law + (size_t)(cnt - (nd + 1)) * V;   // rows for positions P .. P+nd
    const float* dl = nullptr;
    const int32_t* onehot = nullptr;
    if (g.temperature > 0.f && nd > 0) {
        bool any_law = false;
        for (int i = 0; i < nd; ++i) {
            const bool point = g.src[P + i] < 0;
            g.pinned[2 + i] = point ? 1 : 0;
            if (!point) {
                any_law = true;
                CSD_CUDA(cudaMemcpyAsync(g.dl + (size_t)i * V, g.qlaw + (size_t)((P + i) % RING) * V, (size_t)V * 4,
                                         cudaMemcpyDeviceToDevice, g.stream));
            }
        }
        if (any_law) {
            CSD_CUDA(cudaMemcpyAsync(g.onehot_dev, g.pinned + 2, (size_t)nd * 4, cudaMemcpyHostToDevice, g.stream));
            dl = g.dl;
            onehot = g.onehot_dev;
        }
    }
    const float len_r = r == 0 ? 1.f : g.lenience;   // lenience never applies when the target reviews
    volatile int32_t* res = g.pinned;
    res[0] = -1; res[1] = -1;                        // the kernels overwrite both with values >= 0
    csd_status s = csd_spec_accept(target, dl, onehot, g.seq + P, 1, nd, V, g.temperature, len_r, g.seed, g.step++,
                                   g.result_map, g.result_map + 1, g.accept_ws, g.accept_bytes, g.stream);
    if (s != CSD_OK) return s;
    // The accept kernels write (n_acc, out token) straight into mapped pinned host memory.  The host
    // watches the two words instead of sleeping in a stream synchronisation (whose wake-up costs more
    // than the accept call itself) and asks the stream now and then whether it ended early.
    for (unsigned spins = 0; res[0] < 0 || res[1] < 0; ++spins) {
        if ((spins & 0x3ff) == 0x3ff) {
            const cudaError_t q = cudaStreamQuery(g.stream);
            if (q == cudaSuccess) break;             // stream drained: the words are final
            if (q != cudaErrorNotReady) return note_cuda(q);
        }
    }
    if (res[0] < 0 || res[1] < 0) CSD_CUDA(cudaStreamSynchronize(g.stream));
    const int n_acc = g.pinned[0];
    if (n_acc < 0 || n_acc > nd) return CSD_ERR_CUDA;
    g.pinned[CSD_MAX_ROWS + 8] = g.pinned[1];     // (a slot the next review does not overwrite while this copy is in flight)
    CSD_CUDA(cudaMemcpyAsync(g.seq + P + n_acc, g.pinned + CSD_MAX_ROWS + 8, 4, cudaMemcpyHostToDevice, g.stream));
    g.st->reviews[r] += 1;
    g.st->drafted[r] += nd;
    g.st->accepted[r] += n_acc;
    for (int i = 0; i <= n_acc; ++i) {
        g.src[P + i] = (signed char)r;
        if (r > 0 && g.temperature > 0.f)
            CSD_CUDA(cudaMemcpyAsync(g.qlaw + (size_t)((P + i) % RING) * V, target + (size_t)i * V, (size_t)V * 4,
                                     cudaMemcpyDeviceToDevice, g.stream));
    }
    g.len = P + n_acc + 1;
    g.kv[r] = P + n_acc;
    for (int c = r + 1; c < g.n_levels; ++c)
        if (g.kv[c] > P + n_acc) g.kv[c] = P + n_acc;
    return CSD_OK;
}

static csd_status step(Gen& g, int r, int budget) {
    if (r == g.n_levels) {   // base case: the statistical drafter proposes the slot's remaining budget
        if (budget < 1) budget = 1;
        if (g.len + budget > g.cap) return CSD_ERR_CAPACITY;
        csd_status s = g.dynamic ? csd_mag_draft_dynamic(g.mag, g.seq, g.len, g.init_len, budget, g.seq + g.len, g.stream)
                                 : csd_mag_draft(g.mag, g.seq, g.len, budget, g.seq + g.len, g.stream);
        if (s != CSD_OK) return s;
        for (int i = 0; i < budget; ++i) g.src[g.len + i] = -1;
        g.len += budget;
        g.st->mag_calls += 1;
        g.st->mag_tokens += budget;
        return CSD_OK;
    }
    const int P = g.len;
    for (int c = r; c < g.n_levels; ++c) {               // horizontal cascade over the slots
        const int kc = g.K[(size_t)r * g.n_levels + c];
        if (kc <= 0) continue;
        const int start = g.len;
        while (g.len - start < kc) {
            csd_status s = step(g, c + 1, kc - (g.len - start));   // vertical cascade
            if (s != CSD_OK) return s;
        }
    }
    int nd = g.len - P;
    if (nd > g.max_block) nd = g.max_block;              // surplus drafts are dropped
    g.len = P + nd;
    if (P + nd + 1 > g.cap) return CSD_ERR_CAPACITY;
    if (r == 0 && !g.decode_marked) { /* marked by the caller before the first step */ }
    return review(g, r, P, nd);
}

}  // namespace csd

using namespace csd;

extern "C" size_t csd_cascade_workspace_bytes(int vocab, int max_block, int seq_capacity, int haystack_len,
                                              int max_order) {
    if (vocab < 1 || max_block < 0 || max_block > CSD_MAX_ROWS - 1 || seq_capacity < 1 || haystack_len < 0 ||
        max_order < 1 || max_order > CSD_MAG_MAX_ORDER)
        return 0;
    return cascade_layout(vocab, max_block, seq_capacity, haystack_len, max_order).total;
}

extern "C" csd_status csd_cascade_generate(csd_model* const* models, int n_levels, const int32_t* K, int max_block,
                                           float lenience, float temperature, uint64_t seed, int max_order,
                                           int dynamic_haystack, const int32_t* haystack_host, int haystack_len,
                                           const int32_t* bigram_next_dev, const int32_t* init_seq_host, int init_len,
                                           int max_new, int32_t* out_tokens_host, int32_t* out_len,
                                           csd_cascade_stats* stats, void* workspace_dev, size_t workspace_bytes,
                                           void* stream) {
    if (!models || n_levels < 1 || n_levels > 7 || !K || !init_seq_host || init_len < 1 || max_new < 0 ||
        !out_tokens_host || !out_len || !workspace_dev || !bigram_next_dev)
        return CSD_ERR_INVALID_ARG;
    if (max_block < 0 || max_block > CSD_MAX_ROWS - 1 || !(lenience >= 1.f) || !(temperature >= 0.f))
        return CSD_ERR_INVALID_ARG;
    if (max_order < 1 || max_order > CSD_MAG_MAX_ORDER || haystack_len < 0 || (haystack_len > 0 && !haystack_host))
        return CSD_ERR_INVALID_ARG;
    if (((uintptr_t)workspace_dev) & 255) return CSD_ERR_INVALID_ARG;
    const auto t_begin = std::chrono::steady_clock::now();
    *out_len = 0;
    csd_cascade_stats local;
    csd_cascade_stats* st = stats ? stats : &local;
    memset(st, 0, sizeof(*st));
    const long long launches0 = launches_so_far();
    for (int r = 0; r < n_levels; ++r)
        if (!models[r] || models[r]->cfg.vocab != models[0]->cfg.vocab || models[r]->cfg.max_rows < max_block + 1)
            return CSD_ERR_INVALID_ARG;
    Gen g;
    g.models = models; g.n_levels = n_levels; g.K = K; g.max_block = max_block; g.lenience = lenience;
    g.temperature = temperature; g.seed = seed; g.V = models[0]->cfg.vocab; g.st = st;
    g.stream = (cudaStream_t)stream;
    g.dynamic = dynamic_haystack != 0; g.init_len = init_len;
    g.cap = models[0]->cfg.max_seq;
    for (int r = 1; r < n_levels; ++r)
        if (models[r]->cfg.max_seq < g.cap) g.cap = models[r]->cfg.max_seq;
    int window = 0;   // how far drafting can run ahead of the committed prefix
    for (int r = 0; r < n_levels; ++r) {
        for (int c = r; c < n_levels; ++c) window += K[(size_t)r * n_levels + c] > 0 ? K[(size_t)r * n_levels + c] : 0;
        window += max_block + 1;
    }
    if (window >= RING) return CSD_ERR_CAPACITY;
    if (init_len + max_new + window > g.cap) return CSD_ERR_CAPACITY;
    const CascadeWs w = cascade_layout(g.V, max_block, g.cap, haystack_len, max_order);
    if (workspace_bytes < w.total) return CSD_ERR_CAPACITY;
    char* ws = (char*)workspace_dev;
    g.seq = (int32_t*)(ws + w.seq);
    int32_t* hay_dev = (int32_t*)(ws + w.hay);
    g.law = (float*)(ws + w.law); g.qlaw = (float*)(ws + w.qlaw); g.dl = (float*)(ws + w.dl);
    g.onehot_dev = (int32_t*)(ws + w.onehot); g.result_dev = (int32_t*)(ws + w.result);
    g.accept_ws = ws + w.accept; g.accept_bytes = w.total - w.accept;
    g.src.assign((size_t)g.cap + 64, 0);

    HostKit kit;
    {
        const csd_status ks = kit_acquire(kit);
        if (ks != CSD_OK) return ks;
    }
    g.pinned = kit.pinned; g.result_map = kit.mapped;
    cudaEvent_t ev0 = kit.ev[0], ev1 = kit.ev[1], ev2 = kit.ev[2];
    csd_status rc = CSD_OK;
    auto fail = [&](csd_status s) { rc = s; };
    do {
        cudaError_t e = cudaMemcpyAsync(g.seq, init_seq_host, (size_t)init_len * 4, cudaMemcpyHostToDevice, g.stream);
        if (e == cudaSuccess && haystack_len > 0)
            e = cudaMemcpyAsync(hay_dev, haystack_host, (size_t)haystack_len * 4, cudaMemcpyHostToDevice, g.stream);
        if (e == cudaSuccess) e = cudaEventRecord(ev0, g.stream);
        if (e != cudaSuccess) { fail(note_cuda(e)); break; }
        g.len = init_len;
        rc = csd_mag_create(hay_dev, haystack_len, g.V, bigram_next_dev, max_order, 0, ws + w.mag, w.law - w.mag,
                            g.stream, &g.mag);
        if (rc != CSD_OK) break;
        // prefill: encoders (encoder-decoder models), then every prompt token but the last
        for (int r = 0; r < n_levels && rc == CSD_OK; ++r) {
            if (models[r]->cfg.arch == 1) rc = csd_encoder_forward(models[r], hay_dev, haystack_len, g.stream);
            if (rc == CSD_OK && init_len > 1) {
                rc = csd_prefill(models[r], g.seq, init_len - 1, 0, g.stream);
                const int rows = models[r]->cfg.max_rows < CSD_MAX_ROWS ? models[r]->cfg.max_rows : CSD_MAX_ROWS;
                g.st->forwards[r] += (init_len - 1 + rows - 1) / rows;   // counted in review-sized blocks
            }
            g.kv[r] = init_len - 1;
        }
        if (rc != CSD_OK) break;
        if (cudaEventRecord(ev1, g.stream) != cudaSuccess) { fail(note_cuda(cudaGetLastError())); break; }
        while (rc == CSD_OK && g.len - init_len < max_new) rc = step(g, 0, 0);
        if (rc != CSD_OK) break;
        if (cudaEventRecord(ev2, g.stream) != cudaSuccess) { fail(note_cuda(cudaGetLastError())); break; }
        int made = g.len - init_len;
        if (made > max_new) made = max_new;
        if (made > 0) {
            e = cudaMemcpyAsync(out_tokens_host, g.seq + init_len, (size_t)made * 4, cudaMemcpyDeviceToHost, g.stream);
            if (e != cudaSuccess) { fail(note_cuda(e)); break; }
        }
        e = cudaStreamSynchronize(g.stream);
        if (e != cudaSuccess) { fail(note_cuda(e)); break; }
        *out_len = made;
        st->tokens = made;
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, ev0, ev1) == cudaSuccess) st->prefill_ms = ms;
        if (cudaEventElapsedTime(&ms, ev1, ev2) == cudaSuccess) st->decode_ms = ms;
        int code = 0;
        if (csd_device_status(g.stream, &code) == CSD_OK && code != 0) rc = (csd_status)code;
    } while (0);
    if (rc != CSD_OK) cudaStreamSynchronize(g.stream);
    if (g.mag) csd_mag_destroy(g.mag);
    kit_release(kit);
    st->kernel_launches = launches_so_far() - launches0;
    st->total_ms = std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - t_begin).count();
    return rc;
}
