// Multi-Level N-gram module on the GPU (paper Sections 3.1 and 3.2, Algorithm 2).
//
// Per level n two open-addressing hash tables live in device memory (small enough to stay in
// L2): the gram table holds, for every distinct n-gram of the committed tokens, its count and
// last position; the prefix table holds, for every distinct (n-1)-gram context, the successor
// Query would return, packed so that "better" is a plain 64-bit maximum.  Update is two
// order-independent passes (count, then best) built from atomics, so a parallel fold over the
// whole prompt (Initialize) and the fold of a step's few tokens give the state a sequential
// token-by-token Update would give.  All probing is warp-cooperative: the 32 lanes of a warp
// look at 32 consecutive slots at once.
#include "internal.h"

#include <algorithm>
#include <cstring>
#include <map>
#include <new>
#include <vector>

namespace {

constexpr int NG_ERR_FULL = 1;      // probing ran through the whole table
constexpr int NG_ERR_MISSING = 2;   // a gram counted in pass 1 was not found in pass 2
constexpr unsigned FULL_MASK = 0xffffffffu;
constexpr int STEP_THREADS = 1024;

__device__ __forceinline__ unsigned hash_tokens(const int* key, int len) {
    unsigned h = 0x811C9DC5u ^ (unsigned)len;
    for (int i = 0; i < len; ++i) {
        h ^= (unsigned)key[i];
        h *= 0x01000193u;
        h ^= h >> 15;
    }
    h *= 0x85EBCA6Bu;
    h ^= h >> 13;
    h *= 0xC2B2AE35u;
    h ^= h >> 16;
    return h;
}

// Warp-cooperative find (INSERT=false) or find-or-insert (INSERT=true).  `key` holds klen
// tokens; a slot's key is the klen tokens starting at tokens[(ref-1) - n + 1].  Returns the
// slot index, -1 if absent (find only), -2 if the bounded probe ran out.  All 32 lanes call it
// with the same arguments and get the same result.
template <typename Slot, bool INSERT>
__device__ int warp_probe(Slot* table, int cap, const int* tokens, const int* key, int klen,
                          int n, int ref_new) {
    const int lane = threadIdx.x & 31;
    const int mask = cap - 1;
    const int base = (int)(hash_tokens(key, klen) & (unsigned)mask);
    const int windows = cap >> 5;
    int w = 0;
    for (int guard = 0; guard < windows * 33 && w < windows; ++guard) {
        const int slot = (base + w * 32 + lane) & mask;
        const int r = *((volatile int*)&table[slot].ref);
        const bool empty = (r == 0);
        bool match = false;
        if (!empty) {
            const int* sk = tokens + (r - 1) - n + 1;
            match = true;
            for (int i = 0; i < klen; ++i) match = match && (sk[i] == key[i]);
        }
        const unsigned mm = __ballot_sync(FULL_MASK, match);
        const unsigned em = __ballot_sync(FULL_MASK, empty);
        const int fm = mm ? (__ffs(mm) - 1) : 32;
        const int fe = em ? (__ffs(em) - 1) : 32;
        if (fm < fe) return (base + w * 32 + fm) & mask;   // the key sits before the first hole
        if (fe < 32) {
            if (!INSERT) return -1;
            int won = 0;
            if (lane == fe) won = (atomicCAS(&table[slot].ref, 0, ref_new) == 0) ? 1 : 0;
            won = __shfl_sync(FULL_MASK, won, fe);
            if (won) return (base + w * 32 + fe) & mask;
            continue;   // another warp took the hole: look at this window again
        }
        ++w;
    }
    return -2;
}

__device__ __forceinline__ unsigned long long pack_best(int policy, int count, int last, int succ) {
    const unsigned long long c = (policy == 0) ? (unsigned long long)count : 0ull;
    return (c << 44) | ((unsigned long long)last << 24) | (unsigned long long)(unsigned)succ;
}

// Pass 1 for the token at position t, level n: count the n-gram ending at t.
__device__ void fold_count(const NgramDev& c, int t, int n) {
    if (t < n - 1) return;
    const int* key = c.tokens + t - n + 1;
    const int s = warp_probe<GramSlot, true>(c.gram[n], c.cap, c.tokens, key, n, n, t + 1);
    if ((threadIdx.x & 31) == 0) {
        if (s < 0) { atomicExch(&c.state[2], NG_ERR_FULL); return; }
        atomicAdd(&c.gram[n][s].count, 1);
        atomicMax(&c.gram[n][s].last, t);
    }
}

// Pass 2: with every count final, offer this n-gram's (count, last, successor) to its context.
__device__ void fold_best(const NgramDev& c, int t, int n) {
    if (t < n - 1) return;
    const int* key = c.tokens + t - n + 1;
    const int g = warp_probe<GramSlot, false>(c.gram[n], c.cap, c.tokens, key, n, n, 0);
    const int p = warp_probe<PrefSlot, true>(c.pref[n], c.cap, c.tokens, key, n - 1, n, t + 1);
    if ((threadIdx.x & 31) == 0) {
        if (g < 0) { atomicExch(&c.state[2], NG_ERR_MISSING); return; }
        if (p < 0) { atomicExch(&c.state[2], NG_ERR_FULL); return; }
        const int cnt = *((volatile int*)&c.gram[n][g].count), last = *((volatile int*)&c.gram[n][g].last);
        atomicMax(&c.pref[n][p].best, pack_best(c.policy, cnt, last, c.tokens[t]));
    }
}

template <int PASS>
__global__ void ngram_bulk_kernel(NgramDev c, int from, int to) {
    const int levels = c.n_max - c.n_min + 1;
    const int items = (to - from) * levels;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    for (int it = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; it < items; it += warps) {
        const int t = from + it / levels, n = c.n_min + it % levels;
        if (PASS == 1) fold_count(c, t, n); else fold_best(c, t, n);
    }
}

// One block per sequence: fold the tokens committed since the last step (both passes), then
// draft K tokens by chained back-off queries.  Warp w of the first n_max-n_min+1 warps serves
// level n_max - w, so the levels of one query are probed side by side and the longest wins.
__global__ void __launch_bounds__(STEP_THREADS) ngram_step_kernel(const NgramDev* ctxs, SeqState* seqs, int K, int K2) {
    pdl_trigger();
    pdl_wait();
    __shared__ NgramDev c;
    __shared__ int tail[ANPD_N_MAX - 1 + ANPD_K_MAX + 1];
    __shared__ int res[ANPD_N_MAX], res0[ANPD_N_MAX];
    __shared__ int s_avail, s_stop, s_keep;
    if (threadIdx.x == 0) c = ctxs[blockIdx.x];
    __syncthreads();
    SeqState& sq = seqs[blockIdx.x];
    const int from = c.state[1], to = c.state[0];
    const int levels = c.n_max - c.n_min + 1;
    const int warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int items = (to - from) * levels;
    for (int it = warp; it < items; it += nwarps) fold_count(c, from + it / levels, c.n_min + it % levels);
    __threadfence_block();
    __syncthreads();
    for (int it = warp; it < items; it += nwarps) fold_best(c, from + it / levels, c.n_min + it % levels);
    __threadfence_block();
    __syncthreads();

    const int T = to;
    if (threadIdx.x == 0) {
        c.state[1] = to;
        const int keep = min(T, c.n_max - 1);
        for (int i = 0; i < keep; ++i) tail[i] = c.tokens[T - keep + i];
        s_avail = keep;
        s_keep = keep;
        s_stop = (T <= 0 || sq.active == 0) ? 1 : 0;
    }
    __syncthreads();
    int drafted = 0;
    for (int i = 0; i < K; ++i) {
        if (s_stop) break;
        const int avail = s_avail;
        if (warp < levels) {
            const int n = c.n_max - warp, klen = n - 1;
            int ans = -1;
            if (avail >= klen) {
                const int s = warp_probe<PrefSlot, false>(c.pref[n], c.cap, c.tokens, tail + avail - klen, klen, n, 0);
                if (s >= 0) ans = (int)(*((volatile unsigned long long*)&c.pref[n][s].best) & 0xFFFFFFull);
                if (s == -2 && (threadIdx.x & 31) == 0) atomicExch(&c.state[2], NG_ERR_FULL);
            }
            if ((threadIdx.x & 31) == 0) res[warp] = ans;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int ans = -1;
            for (int w = 0; w < levels && ans < 0; ++w) ans = res[w];   // longest level first
            if (i == 0) for (int w = 0; w < levels; ++w) res0[w] = res[w];
            if (ans < 0) s_stop = 1;
            else { tail[avail] = ans; s_avail = avail + 1; sq.draft[i] = ans; }
        }
        __syncthreads();
        if (!s_stop) ++drafted;
    }
    if (threadIdx.x == 0) {
        sq.draft_len = drafted;
        sq.last_tok = (T > 0) ? c.tokens[T - 1] : 0;
    }
    // The second candidate: its first token is the answer of the longest level that disagrees with the first candidate's
    // first token; it then continues like the first one, by back-off queries on its own temporary context.
    int drafted2 = 0;
    if (K2 > 0 && drafted > 0) {
        __syncthreads();
        if (threadIdx.x == 0) {
            int alt = -1;
            for (int w = 0; w < levels && alt < 0; ++w)
                if (res0[w] >= 0 && res0[w] != sq.draft[0]) alt = res0[w];
            s_stop = alt < 0 ? 1 : 0;
            if (alt >= 0) { tail[s_keep] = alt; s_avail = s_keep + 1; sq.draft2[0] = alt; }
        }
        __syncthreads();
        if (!s_stop) drafted2 = 1;
        for (int i = 1; i < K2; ++i) {
            if (s_stop) break;
            const int avail = s_avail;
            if (warp < levels) {
                const int n = c.n_max - warp, klen = n - 1;
                int ans = -1;
                if (avail >= klen) {
                    const int s = warp_probe<PrefSlot, false>(c.pref[n], c.cap, c.tokens, tail + avail - klen, klen, n, 0);
                    if (s >= 0) ans = (int)(*((volatile unsigned long long*)&c.pref[n][s].best) & 0xFFFFFFull);
                    if (s == -2 && (threadIdx.x & 31) == 0) atomicExch(&c.state[2], NG_ERR_FULL);
                }
                if ((threadIdx.x & 31) == 0) res[warp] = ans;
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                int ans = -1;
                for (int w = 0; w < levels && ans < 0; ++w) ans = res[w];
                if (ans < 0) s_stop = 1;
                else { tail[avail] = ans; s_avail = avail + 1; sq.draft2[i] = ans; }
            }
            __syncthreads();
            if (!s_stop) ++drafted2;
        }
    }
    if (threadIdx.x == 0) sq.draft2_len = drafted2;
}

int next_pow2(int v) { int p = 64; while (p < v) p <<= 1; return p; }

}  // namespace

anpd_status ngram_enqueue_bulk(anpd_ngram* ctx, int from, int to, Profiler* prof, cudaStream_t on) {
    if (to <= from) return ANPD_OK;
    cudaStream_t st = on ? on : ctx->stream;
    const int levels = ctx->h.n_max - ctx->h.n_min + 1;
    const int items = (to - from) * levels;
    const int threads = 256, wpb = threads / 32;
    const int blocks = std::min((items + wpb - 1) / wpb, 148 * 8);
    LAUNCH(prof, st, KC_NGRAM, 0, (ngram_bulk_kernel<1><<<blocks, threads, 0, st>>>(ctx->h, from, to)));
    LAUNCH(prof, st, KC_NGRAM, 0, (ngram_bulk_kernel<2><<<blocks, threads, 0, st>>>(ctx->h, from, to)));
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}

anpd_status ngram_enqueue_step(const NgramDev* d_ctxs, SeqState* d_seq, int batch, int K,
                               cudaStream_t st, Profiler* prof, int K2) {
    LAUNCH(prof, st, KC_NGRAM, 0, (launch_k(ngram_step_kernel, batch, STEP_THREADS, 0, st, d_ctxs, d_seq, K, K2)));
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}

// ---------------------------------------------------------------------------------------------
// boundary
// ---------------------------------------------------------------------------------------------
extern "C" {

anpd_status anpd_ngram_create(const anpd_ngram_config* cfg, void* cuda_stream, anpd_ngram** out) {
    if (!cfg || !out) return ANPD_ERR_ARG;
    if (cfg->n_min < 2 || cfg->n_max < cfg->n_min || cfg->n_max > ANPD_N_MAX) return ANPD_ERR_RANGE;
    if (cfg->max_ctx < 1 || cfg->max_ctx > (1 << 20)) return ANPD_ERR_ARG;
    if (cfg->policy != 0 && cfg->policy != 1) return ANPD_ERR_ARG;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) { cudaGetLastError(); return ANPD_ERR_CUDA; }
    anpd_ngram* c = new (std::nothrow) anpd_ngram();
    if (!c) return ANPD_ERR_OOM;
    std::memset(&c->h, 0, sizeof(c->h));
    c->d = nullptr; c->pinned = nullptr; c->slab = nullptr; c->n_tokens = 0; c->n_folded = 0;
    c->stream = (cudaStream_t)cuda_stream;
    const int cap = next_pow2(2 * cfg->max_ctx);
    const int levels = cfg->n_max - cfg->n_min + 1;
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    const size_t tok_b = up(sizeof(int) * (size_t)cfg->max_ctx), st_b = 256, seq_b = up(sizeof(SeqState));
    const size_t gram_b = up(sizeof(GramSlot) * (size_t)cap), pref_b = up(sizeof(PrefSlot) * (size_t)cap);
    c->slab_bytes = tok_b + st_b + seq_b + up(sizeof(NgramDev)) + levels * (gram_b + pref_b);
    if (cudaMalloc(&c->slab, c->slab_bytes) != cudaSuccess) { cudaGetLastError(); delete c; return ANPD_ERR_OOM; }
    if (cudaMallocHost((void**)&c->pinned, 256) != cudaSuccess) { cudaGetLastError(); cudaFree(c->slab); delete c; return ANPD_ERR_OOM; }
    char* p = (char*)c->slab;
    c->h.tokens = (int*)p; p += tok_b;
    c->h.state = (int*)p; p += st_b;
    p += seq_b;                                   // a SeqState used by anpd_ngram_draft
    c->d = (NgramDev*)p; p += up(sizeof(NgramDev));
    for (int n = cfg->n_min; n <= cfg->n_max; ++n) {
        c->h.gram[n] = (GramSlot*)p; p += gram_b;
        c->h.pref[n] = (PrefSlot*)p; p += pref_b;
    }
    c->h.n_min = cfg->n_min; c->h.n_max = cfg->n_max; c->h.max_ctx = cfg->max_ctx;
    c->h.cap = cap; c->h.policy = cfg->policy;
    if (cudaMemsetAsync(c->slab, 0, c->slab_bytes, c->stream) != cudaSuccess ||
        cudaMemcpyAsync(c->d, &c->h, sizeof(NgramDev), cudaMemcpyHostToDevice, c->stream) != cudaSuccess ||
        cudaStreamSynchronize(c->stream) != cudaSuccess) {
        anpd_note_cuda_error(cudaGetLastError(), __FILE__, __LINE__);
        cudaFreeHost(c->pinned); cudaFree(c->slab); delete c;
        return ANPD_ERR_CUDA;
    }
    *out = c;
    return ANPD_OK;
}

anpd_status anpd_ngram_reset(anpd_ngram* c) {
    if (!c) return ANPD_ERR_ARG;
    CUDA_TRY(cudaMemsetAsync(c->slab, 0, c->slab_bytes, c->stream));
    CUDA_TRY(cudaMemcpyAsync(c->d, &c->h, sizeof(NgramDev), cudaMemcpyHostToDevice, c->stream));
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    c->n_tokens = 0;
    c->n_folded = 0;
    return ANPD_OK;
}

anpd_status anpd_ngram_destroy(anpd_ngram* c) {
    if (!c) return ANPD_ERR_ARG;
    cudaStreamSynchronize(c->stream);
    cudaFreeHost(c->pinned);
    cudaFree(c->slab);
    delete c;
    return ANPD_OK;
}

anpd_status anpd_ngram_len(anpd_ngram* c, int* n_tokens) {
    if (!c || !n_tokens) return ANPD_ERR_ARG;
    *n_tokens = c->n_tokens;
    return ANPD_OK;
}

anpd_status anpd_ngram_update(anpd_ngram* c, const int32_t* new_tokens, int n_new) {
    if (!c || (n_new > 0 && !new_tokens) || n_new < 0) return ANPD_ERR_ARG;
    if (n_new == 0) return ANPD_OK;
    for (int i = 0; i < n_new; ++i)
        if (new_tokens[i] < 0 || new_tokens[i] >= (1 << 24)) return ANPD_ERR_RANGE;
    if (c->n_tokens + n_new > c->h.max_ctx) return ANPD_ERR_CAPACITY;
    const int from = c->n_tokens, to = from + n_new;
    CUDA_TRY(cudaMemcpyAsync(c->h.tokens + from, new_tokens, sizeof(int) * (size_t)n_new, cudaMemcpyHostToDevice, c->stream));
    c->pinned[0] = to; c->pinned[1] = to;
    CUDA_TRY(cudaMemcpyAsync(c->h.state, c->pinned, 2 * sizeof(int), cudaMemcpyHostToDevice, c->stream));
    // tokens a decoding loop committed in its last step are still waiting to be folded
    ANPD_TRY(ngram_enqueue_bulk(c, c->n_folded, to, nullptr));
    CUDA_TRY(cudaMemcpyAsync(c->pinned + 8, c->h.state + 2, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    c->n_tokens = to;
    c->n_folded = to;
    return c->pinned[8] == 0 ? ANPD_OK : ANPD_ERR_CUDA;
}

anpd_status anpd_ngram_draft(anpd_ngram* c, int K, int32_t* draft, int* draft_len) {
    if (!c || !draft_len || (K > 0 && !draft)) return ANPD_ERR_ARG;
    if (K < 0 || K > ANPD_K_MAX) return ANPD_ERR_RANGE;
    if (c->n_tokens < 1) return ANPD_ERR_STATE;
    SeqState* d_seq = (SeqState*)((char*)c->h.state + 256);
    // active = 1, everything else 0
    SeqState init; std::memset(&init, 0, sizeof(init)); init.active = 1;
    std::memcpy(c->pinned + 16, &init, sizeof(init));
    static_assert(sizeof(SeqState) <= 256 - 64, "staging buffer too small");
    CUDA_TRY(cudaMemcpyAsync(d_seq, c->pinned + 16, sizeof(SeqState), cudaMemcpyHostToDevice, c->stream));
    ANPD_TRY(ngram_enqueue_step(c->d, d_seq, 1, K, c->stream, nullptr));
    CUDA_TRY(cudaMemcpyAsync(c->pinned + 16, d_seq, sizeof(SeqState), cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(cudaMemcpyAsync(c->pinned + 8, c->h.state + 2, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    if (c->pinned[8] != 0) return ANPD_ERR_CUDA;
    c->n_folded = c->n_tokens;
    SeqState got; std::memcpy(&got, c->pinned + 16, sizeof(got));
    for (int i = 0; i < got.draft_len; ++i) draft[i] = got.draft[i];
    *draft_len = got.draft_len;
    return ANPD_OK;
}

static anpd_status dump_level(anpd_ngram* c, int n, std::vector<anpd_ngram_entry>& grams,
                              std::vector<anpd_ngram_entry>* bests) {
    if (n < c->h.n_min || n > c->h.n_max) return ANPD_ERR_RANGE;
    std::vector<int> tok((size_t)std::max(c->n_tokens, 1));
    std::vector<GramSlot> g((size_t)c->h.cap);
    std::vector<PrefSlot> p((size_t)c->h.cap);
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    if (c->n_tokens > 0) CUDA_TRY(cudaMemcpy(tok.data(), c->h.tokens, sizeof(int) * (size_t)c->n_tokens, cudaMemcpyDeviceToHost));
    CUDA_TRY(cudaMemcpy(g.data(), c->h.gram[n], sizeof(GramSlot) * g.size(), cudaMemcpyDeviceToHost));
    CUDA_TRY(cudaMemcpy(p.data(), c->h.pref[n], sizeof(PrefSlot) * p.size(), cudaMemcpyDeviceToHost));
    auto less = [](const anpd_ngram_entry& a, const anpd_ngram_entry& b) {
        for (int i = 0; i < ANPD_N_MAX - 1; ++i) if (a.key[i] != b.key[i]) return a.key[i] < b.key[i];
        return a.succ < b.succ;
    };
    grams.clear();
    for (const GramSlot& s : g) {
        if (s.ref == 0) continue;
        anpd_ngram_entry e;
        const int t = s.ref - 1;
        for (int i = 0; i < ANPD_N_MAX - 1; ++i) e.key[i] = (i < n - 1) ? tok[t - n + 1 + i] : -1;
        e.succ = tok[t]; e.count = s.count; e.last_pos = s.last;
        grams.push_back(e);
    }
    std::sort(grams.begin(), grams.end(), less);
    if (bests) {
        bests->clear();
        for (const PrefSlot& s : p) {
            if (s.ref == 0) continue;
            anpd_ngram_entry e;
            const int t = s.ref - 1;
            for (int i = 0; i < ANPD_N_MAX - 1; ++i) e.key[i] = (i < n - 1) ? tok[t - n + 1 + i] : -1;
            e.succ = (int)(s.best & 0xFFFFFFull);
            e.last_pos = (int)((s.best >> 24) & 0xFFFFFull);
            e.count = 0;
            auto it = std::lower_bound(grams.begin(), grams.end(), e, less);
            if (it != grams.end() && !less(e, *it)) e.count = it->count;
            bests->push_back(e);
        }
        std::sort(bests->begin(), bests->end(), less);
    }
    return ANPD_OK;
}

anpd_status anpd_ngram_dump(anpd_ngram* c, int n, anpd_ngram_entry* out, int cap, int* n_entries) {
    if (!c || !n_entries) return ANPD_ERR_ARG;
    std::vector<anpd_ngram_entry> grams;
    ANPD_TRY(dump_level(c, n, grams, nullptr));
    if (out) {
        if ((int)grams.size() > cap) return ANPD_ERR_CAPACITY;
        std::copy(grams.begin(), grams.end(), out);
    }
    *n_entries = (int)grams.size();
    return ANPD_OK;
}

anpd_status anpd_ngram_dump_best(anpd_ngram* c, int n, anpd_ngram_entry* out, int cap, int* n_entries) {
    if (!c || !n_entries) return ANPD_ERR_ARG;
    std::vector<anpd_ngram_entry> grams, bests;
    ANPD_TRY(dump_level(c, n, grams, &bests));
    if (out) {
        if ((int)bests.size() > cap) return ANPD_ERR_CAPACITY;
        std::copy(bests.begin(), bests.end(), out);
    }
    *n_entries = (int)bests.size();
    return ANPD_OK;
}

}  // extern "C"
