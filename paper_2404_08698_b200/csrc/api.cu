// Handles, the verify / prefill / generate entry points and the measurement hooks.
#include "internal.h"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

typedef __nv_bfloat16 bf16;

std::atomic<long long> g_launch_count{0};
const bool g_use_pdl = std::getenv("ANPD_NO_PDL") == nullptr;
thread_local bool t_no_pdl = false;
// text of the calling thread's last CUDA failure (anpd_status_string(ANPD_ERR_CUDA) returns it)
static thread_local char g_last_error[256] = "";

void anpd_note_cuda_error(cudaError_t e, const char* file, int line) {
    std::snprintf(g_last_error, sizeof(g_last_error), "%s at %s:%d", cudaGetErrorString(e), file, line);
    if (std::getenv("ANPD_VERBOSE")) std::fprintf(stderr, "[anpd] CUDA error: %s\n", g_last_error);
    cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// profiler
// ---------------------------------------------------------------------------------------------
void Profiler::begin(cudaStream_t st, int c, double b) {
    if (used * 2 + 2 > ev.size()) {
        for (int i = 0; i < 2; ++i) { cudaEvent_t e; cudaEventCreate(&e); ev.push_back(e); }
        cls.push_back(0); bytes.push_back(0);
    }
    cls[used] = c; bytes[used] = b;
    cudaEventRecord(ev[used * 2], st);
}
void Profiler::end(cudaStream_t st) {
    cudaEventRecord(ev[used * 2 + 1], st);
    ++used;
}
void Profiler::drain() {
    for (size_t i = 0; i < used; ++i) {
        cudaEventSynchronize(ev[i * 2 + 1]);
        float t = 0;
        if (cudaEventElapsedTime(&t, ev[i * 2], ev[i * 2 + 1]) == cudaSuccess) {
            ms[cls[i]] += t; n[cls[i]] += 1;
            if (cls[i] == KC_GEMM) gemm_bytes += bytes[i];
        }
    }
    used = 0;
}
void Profiler::clear() {
    used = 0; gemm_bytes = 0;
    for (int i = 0; i < KC_COUNT; ++i) { ms[i] = 0; n[i] = 0; }
}
Profiler::~Profiler() { for (cudaEvent_t e : ev) cudaEventDestroy(e); }

namespace {

__global__ void f32_to_bf16_kernel(const float* __restrict__ src, bf16* __restrict__ dst, size_t n) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        dst[i] = __float2bfloat16_rn(src[i]);
}
__global__ void set_int_kernel(int* p, int v) { *p = v; }
// A sequence that starts over: empty cache, counters cleared, active (a finished decoding loop leaves it retired).
__global__ void seq_restart_kernel(SeqState* s) {
    s->kv_len = 0; s->draft_len = 0; s->accepted_len = 0;
    s->steps = 0; s->drafted = 0; s->accepted = 0;
    s->draft2_len = 0; s->alt_wins = 0; s->move_n = 0;
    for (int i = 0; i < 8; ++i) s->hist[i] = 0;
    s->active = 1; s->stop_at = 0x7fffffff; s->error = 0;
}
__global__ void greedy_stage_kernel(SeqState* seqs) {
    pdl_trigger();
    pdl_wait();
    SeqState& s = seqs[blockIdx.x];
    s.last_tok = s.next_tok;
    s.draft_len = 0;
    s.draft2_len = 0;
}

// Last kernel of a step inside the device-resident decoding loop: the loop goes on while a sequence is still active and
// nothing has failed (a sequence's sticky error, a kernel that gave up waiting, more steps than the caller allowed).
__global__ void loop_condition_kernel(const SeqState* seqs, int batch, const int* kernel_err, int* steps_left, cudaGraphConditionalHandle handle) {
    pdl_trigger();
    pdl_wait();
    if (threadIdx.x != 0) return;
    bool go = false;
    for (int b = 0; b < batch; ++b) {
        if (seqs[b].error != 0) { go = false; break; }
        go = go || seqs[b].active != 0;
    }
    if (*kernel_err != 0) go = false;
    const int left = *steps_left - 1;
    *steps_left = left;
    if (left <= 0) go = false;
    cudaGraphSetConditional(handle, go ? 1u : 0u);
}

inline size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }

uint16_t f32_to_bf16_host(float f) {
    uint32_t u; std::memcpy(&u, &f, 4);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

// Copies one tensor into library memory as bf16 (matrices) or fp32 (norm gains).
anpd_status upload(void* dst, const void* src, size_t n, bool as_bf16, bool src_bf16, bool on_device, cudaStream_t st,
                   std::vector<uint16_t>& tmp, float* d_tmp, size_t d_tmp_elems) {
    if (!as_bf16) {
        CUDA_TRY(cudaMemcpyAsync(dst, src, n * 4, on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, st));
        return ANPD_OK;
    }
    if (src_bf16) {
        CUDA_TRY(cudaMemcpyAsync(dst, src, n * 2, on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, st));
        if (!on_device) CUDA_TRY(cudaStreamSynchronize(st));
        return ANPD_OK;
    }
    if (on_device) {
        LAUNCH(nullptr, st, KC_OTHER, 0, (f32_to_bf16_kernel<<<1024, 256, 0, st>>>((const float*)src, (bf16*)dst, n)));
        CUDA_TRY(cudaGetLastError());
        return ANPD_OK;
    }
    (void)d_tmp; (void)d_tmp_elems;
    tmp.resize(n);
    const float* f = (const float*)src;
    for (size_t i = 0; i < n; ++i) tmp[i] = f32_to_bf16_host(f[i]);
    CUDA_TRY(cudaMemcpyAsync(dst, tmp.data(), n * 2, cudaMemcpyHostToDevice, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    return ANPD_OK;
}

// The model's weight blocks are ordered for the SM count of the device it was created on, and its
// memory lives there: refuse to run with another device current.
anpd_status check_device(const anpd_model* m) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return ANPD_ERR_CUDA; }
    return dev == m->device ? ANPD_OK : ANPD_ERR_STATE;
}

bool have_device() {
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess || n == 0) { cudaGetLastError(); return false; }
    return true;
}

}  // namespace

// GEMM plans (how each matrix shape is cut across the SMs) and the TMA views of the weights.
static anpd_status model_make_plans(anpd_model* m) {
    const anpd_model_config& c = m->cfg;
    m->plain_gemm = std::getenv("ANPD_PLAIN_GEMM") != nullptr;
    size_t ints = 0;
    int max_tiles = 0;
    m->max_segs = 1;
    for (int k = 0; k < GK_COUNT; ++k) {
        ints += 2 * (size_t)m->plan[k].m_tiles;
        max_tiles = std::max(max_tiles, m->plan[k].m_tiles);
        m->max_segs = std::max(m->max_segs, m->plan[k].max_segs);
    }
    ints += 4 * (size_t)max_tiles + (size_t)GK_COUNT * max_tiles;
    std::vector<int> host(ints);
    CUDA_TRY(cudaMalloc((void**)&m->d_plan_tables, ints * sizeof(int)));
    size_t off = 0;
    for (int k = 0; k < GK_COUNT; ++k) {
        GemmPlan& p = m->plan[k];
        p.d_first_cta = m->d_plan_tables + off;
        std::copy(p.first_cta.begin(), p.first_cta.end(), host.begin() + off); off += p.m_tiles;
        p.d_seg_count = m->d_plan_tables + off;
        std::copy(p.seg_count.begin(), p.seg_count.end(), host.begin() + off); off += p.m_tiles;
    }
    m->d_ones = m->d_plan_tables + off;
    for (int i = 0; i < max_tiles; ++i) host[off + i] = 1;
    m->d_const_segs[0] = m->d_const_segs[1] = m->d_ones;
    for (int k = 2; k <= 3; ++k) {
        m->d_const_segs[k] = m->d_plan_tables + off + (size_t)(k - 1) * max_tiles;
        for (int i = 0; i < max_tiles; ++i) host[off + (size_t)(k - 1) * max_tiles + i] = k;
    }
    for (int k = 0; k < GK_COUNT; ++k) {
        m->d_tail_segs[k] = m->d_plan_tables + off + (size_t)(3 + k) * max_tiles;
        m->tail_cfg[k] = -1;
    }
    CUDA_TRY(cudaMemcpy(m->d_plan_tables, host.data(), ints * sizeof(int), cudaMemcpyHostToDevice));
    return ANPD_OK;
}

extern "C" {

const char* anpd_status_string(anpd_status s) {
    switch (s) {
        case ANPD_OK: return "ok";
        case ANPD_ERR_ARG: return "bad argument";
        case ANPD_ERR_OOM: return "out of memory";
        case ANPD_ERR_CAPACITY: return "capacity exceeded";
        case ANPD_ERR_RANGE: return "value out of range";
        case ANPD_ERR_CUDA: return g_last_error[0] ? g_last_error : "CUDA error";
        case ANPD_ERR_STATE: return "call out of order";
        default: return "unknown status";
    }
}

long long anpd_launch_count(int reset) {
    return reset ? g_launch_count.exchange(0) : g_launch_count.load();
}

// ---------------------------------------------------------------------------------------------
// model
// ---------------------------------------------------------------------------------------------
anpd_status anpd_model_create(const anpd_model_config* cfg, const void* const* weights, int weights_are_bf16,
                              int weights_on_device, void* cuda_stream, anpd_model** out) {
    if (!cfg || !weights || !out) return ANPD_ERR_ARG;
    const anpd_model_config& c = *cfg;
    if (c.n_layers < 1 || c.d_model < 8 || c.n_q_heads < 1 || c.n_kv_heads < 1 || c.d_ffn < 8 || c.vocab < 1) return ANPD_ERR_ARG;
    if (c.head_dim != 64 && c.head_dim != 128) return ANPD_ERR_ARG;
    {
        const int grp = c.n_q_heads / c.n_kv_heads;          // query heads per kv head
        if (c.n_q_heads % c.n_kv_heads != 0 || (grp != 1 && grp != 2 && grp != 4 && grp != 8)) return ANPD_ERR_ARG;
    }
    if (c.d_model > 16384) return ANPD_ERR_ARG;
    if (c.d_model % 8 || c.d_ffn % 8 || c.vocab >= (1 << 24)) return ANPD_ERR_ARG;
    if (!(c.rope_theta > 0.0f) || !(c.rms_eps >= 0.0f)) return ANPD_ERR_ARG;
    const int n_tensors = 1 + 9 * c.n_layers + 2;
    for (int i = 0; i < n_tensors; ++i) if (!weights[i]) return ANPD_ERR_ARG;
    if (!have_device()) return ANPD_ERR_CUDA;

    anpd_model* m = new (std::nothrow) anpd_model();
    if (!m) return ANPD_ERR_OOM;
    m->cfg = c;
    m->stream = (cudaStream_t)cuda_stream;
    m->dq = c.n_q_heads * c.head_dim;
    m->dkv = c.n_kv_heads * c.head_dim;
    m->nqkv = m->dq + 2 * m->dkv;
    const size_t d = c.d_model, F = c.d_ffn, V = c.vocab;
    // GEMM weights are stored tile by tile (128 output rows x 64 inputs, 16 KB contiguous each, zero
    // padded at ragged edges) so that every TMA box is one contiguous read; the embedding table stays
    // row-major because it is only gathered.
    {
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            cudaGetLastError(); delete m; return ANPD_ERR_CUDA;
        }
        m->num_sms = sms;
        m->device = dev;
        const int shapes[GK_COUNT][2] = {{m->nqkv, c.d_model}, {c.d_model, m->dq}, {2 * c.d_ffn, c.d_model}, {c.d_model, c.d_ffn},
                                         {c.vocab, c.d_model}};
        for (int k = 0; k < GK_COUNT; ++k) gemm_make_plan(&m->plan[k], shapes[k][0], shapes[k][1], sms);
        for (int k = 0; k < GK_COUNT; ++k) rr_make_plan(&m->rr[k], shapes[k][0], shapes[k][1], sms);
    }
    m->rr_slab = nullptr;
    m->rr_lm = nullptr;
    // ANPD_RR=1: single-sequence steps run on a second copy of the projections in row-range storage (proj_rr.cu).  Off
    // by default: measured at every model shape, the fused epilogues cost more than the small kernels they replace.
    m->rr_ready = std::getenv("ANPD_RR") != nullptr;
    for (int k = 0; k < GK_COUNT; ++k)
        if (m->rr[k].mt > 2) m->rr_ready = false;      // a CTA's feature range must fit two 128-row MMA tiles (very large vocabularies do not)
    const size_t b_embed = up256(V * d * 2), b_lm = up256(gemm_tiled_elems(m->plan[GK_LM]) * 2),
                 b_qkv = up256(gemm_tiled_elems(m->plan[GK_QKV]) * 2), b_o = up256(gemm_tiled_elems(m->plan[GK_O]) * 2),
                 b_gu = up256(gemm_tiled_elems(m->plan[GK_GU]) * 2), b_d = up256(gemm_tiled_elems(m->plan[GK_DOWN]) * 2),
                 b_norm = up256(d * 4);
    m->slab_bytes = b_embed + b_lm + b_norm + c.n_layers * (b_qkv + b_o + b_gu + b_d + 2 * b_norm);
    if (cudaMalloc(&m->slab, m->slab_bytes) != cudaSuccess) { cudaGetLastError(); delete m; return ANPD_ERR_OOM; }
    size_t rr_bytes[GK_COUNT], rr_total = 0;
    for (int k = 0; k < GK_COUNT; ++k) {
        rr_bytes[k] = up256(rr_storage_bytes(m->rr[k]));
        rr_total += rr_bytes[k] * (k == GK_LM ? 1 : (size_t)c.n_layers);
    }
    if (m->rr_ready && cudaMalloc(&m->rr_slab, rr_total) != cudaSuccess) { cudaGetLastError(); cudaFree(m->slab); delete m; return ANPD_ERR_OOM; }
    m->streamed_bytes = 2.0 * ((double)c.n_layers * ((double)m->nqkv * d + (double)d * m->dq + 3.0 * F * d) + (double)V * d);

    char* p = (char*)m->slab;
    std::vector<uint16_t> tmp;
    const bool bf = weights_are_bf16 != 0, dev = weights_on_device != 0;
    cudaStream_t st = m->stream;
    anpd_status rc = ANPD_OK;
    // staging for host-side sources: the largest matrix in its source type
    void* stage = nullptr;
    const size_t max_elems = std::max(std::max((size_t)V * d, F * d), std::max((size_t)m->dq * d, d * F));
    if (!dev && cudaMalloc(&stage, max_elems * (bf ? 2 : 4)) != cudaSuccess) { cudaGetLastError(); cudaFree(m->rr_slab); cudaFree(m->slab); delete m; return ANPD_ERR_OOM; }
    if (cudaMemsetAsync(m->slab, 0, m->slab_bytes, st) != cudaSuccess) rc = ANPD_ERR_CUDA;
    if (m->rr_ready && cudaMemsetAsync(m->rr_slab, 0, rr_total, st) != cudaSuccess) rc = ANPD_ERR_CUDA;
    unsigned char* rp = (unsigned char*)m->rr_slab;     // next free byte of the row-range storage
    auto put = [&](const void* src, size_t n, bool as_bf16, size_t bytes) -> void* {
        void* dst = p;
        p += bytes;
        if (rc == ANPD_OK) rc = upload(dst, src, n, as_bf16, bf, dev, st, tmp, nullptr, 0);
        return dst;
    };
    // rows [row_off, row_off + rows) of a tiled [*, K] matrix at dst, and of its row-range copy at rdst
    auto put_tiled = [&](int kind, const void* src, int rows, int K, int row_off, void* dst, unsigned char* rdst) {
        if (rc != ANPD_OK) return;
        const void* dsrc = src;
        if (!dev) {
            if (cudaMemcpyAsync(stage, src, (size_t)rows * K * (bf ? 2 : 4), cudaMemcpyHostToDevice, st) != cudaSuccess ||
                cudaStreamSynchronize(st) != cudaSuccess) { anpd_note_cuda_error(cudaGetLastError(), __FILE__, __LINE__); rc = ANPD_ERR_CUDA; return; }
            dsrc = stage;
        }
        rc = gemm_retile_enqueue(m->plan[kind], dsrc, !bf, rows, row_off, (bf16*)dst, st);
        if (rc == ANPD_OK && m->rr_ready) {
            const int map = kind == GK_QKV ? RR_MAP_HEADS : kind == GK_GU ? RR_MAP_GATE_UP : RR_MAP_IDENTITY;
            rc = rr_retile_enqueue(m->rr[kind], dsrc, !bf, rows, row_off, map, c.head_dim, c.d_ffn, rdst, st);
        }
        if (rc == ANPD_OK && !dev && cudaStreamSynchronize(st) != cudaSuccess) { anpd_note_cuda_error(cudaGetLastError(), __FILE__, __LINE__); rc = ANPD_ERR_CUDA; }
    };
    int t = 0;
    m->embed = (const bf16*)put(weights[t++], V * d, true, b_embed);
    m->layers.resize(c.n_layers);
    m->rr_layers.resize(c.n_layers);
    for (int l = 0; l < c.n_layers; ++l) {
        LayerW& w = m->layers[l];
        anpd_model::LayerRR& r = m->rr_layers[l];
        w.attn_norm = (const float*)put(weights[t++], d, false, b_norm);
        // q, k and v rows form one matrix so that one GEMM produces all three
        w.wqkv = (const bf16*)p;
        r.wqkv = rp;
        put_tiled(GK_QKV, weights[t++], m->dq, (int)d, 0, p, rp);
        put_tiled(GK_QKV, weights[t++], m->dkv, (int)d, m->dq, p, rp);
        put_tiled(GK_QKV, weights[t++], m->dkv, (int)d, m->dq + m->dkv, p, rp);
        p += b_qkv; rp += rr_bytes[GK_QKV];
        w.wo = (const bf16*)p;
        r.wo = rp;
        put_tiled(GK_O, weights[t++], (int)d, m->dq, 0, p, rp);
        p += b_o; rp += rr_bytes[GK_O];
        w.ffn_norm = (const float*)put(weights[t++], d, false, b_norm);
        w.wgu = (const bf16*)p;
        r.wgu = rp;
        put_tiled(GK_GU, weights[t++], (int)F, (int)d, 0, p, rp);
        put_tiled(GK_GU, weights[t++], (int)F, (int)d, (int)F, p, rp);
        p += b_gu; rp += rr_bytes[GK_GU];
        w.wd = (const bf16*)p;
        r.wd = rp;
        put_tiled(GK_DOWN, weights[t++], (int)d, (int)F, 0, p, rp);
        p += b_d; rp += rr_bytes[GK_DOWN];
    }
    m->final_norm = (const float*)put(weights[t++], d, false, b_norm);
    m->lm_head = (const bf16*)p;
    m->rr_lm = rp;
    put_tiled(GK_LM, weights[t++], (int)V, (int)d, 0, p, rp);
    p += b_lm;
    if (rc == ANPD_OK && cudaStreamSynchronize(st) != cudaSuccess) { anpd_note_cuda_error(cudaGetLastError(), __FILE__, __LINE__); rc = ANPD_ERR_CUDA; }
    if (stage) cudaFree(stage);
    m->d_plan_tables = nullptr;
    if (rc == ANPD_OK) rc = model_make_plans(m);
    if (rc != ANPD_OK) { cudaFree(m->d_plan_tables); cudaFree(m->rr_slab); cudaFree(m->slab); delete m; return rc; }
    *out = m;
    return ANPD_OK;
}

anpd_status anpd_model_destroy(anpd_model* m) {
    if (!m) return ANPD_ERR_ARG;
    cudaStreamSynchronize(m->stream);
    cudaFree(m->d_plan_tables);
    cudaFree(m->rr_slab);
    cudaFree(m->slab);
    delete m;
    return ANPD_OK;
}

// ---------------------------------------------------------------------------------------------
// KV cache + workspace
// ---------------------------------------------------------------------------------------------
anpd_status anpd_kv_create(const anpd_model* cm, int max_len, int batch, int shuffle_pages, anpd_kv** out) {
    if (!cm || !out || max_len < ANPD_ROWS || max_len > 256 * KV_PAGE || batch < 1 || batch > 16) return ANPD_ERR_ARG;
    anpd_model* m = const_cast<anpd_model*>(cm);
    const anpd_model_config& c = m->cfg;
    anpd_kv* kv = new (std::nothrow) anpd_kv();
    if (!kv) return ANPD_ERR_OOM;
    kv->m = m; kv->batch = batch;
    kv->pages_per_seq = (max_len + KV_PAGE - 1) / KV_PAGE;
    kv->max_len = kv->pages_per_seq * KV_PAGE;
    kv->total_pages = kv->pages_per_seq * batch;
    kv->staged = false;
    kv->candidates = 1;
    kv->warm = false;
    kv->loop_ok = std::getenv("ANPD_HOST_LOOP") == nullptr;
    kv->side_stream = nullptr; kv->ev_fork = nullptr; kv->ev_join = nullptr;
    if (!m->prof.on && cudaStreamCreateWithFlags(&kv->side_stream, cudaStreamNonBlocking) == cudaSuccess) {
        if (cudaEventCreateWithFlags(&kv->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&kv->ev_join, cudaEventDisableTiming) != cudaSuccess) {
            cudaGetLastError();
            if (kv->ev_fork) cudaEventDestroy(kv->ev_fork);
            cudaStreamDestroy(kv->side_stream);
            kv->side_stream = nullptr; kv->ev_fork = nullptr; kv->ev_join = nullptr;
        }
    } else cudaGetLastError();
    kv->loop_launches_per_step = 0;
    // the legacy default stream cannot be captured: steps on it are launched one kernel at a time
    kv->use_graphs = std::getenv("ANPD_NO_GRAPH") == nullptr && m->stream != nullptr && m->stream != cudaStreamLegacy;
    kv->h_kv_len.assign(batch, 0);
    kv->h_len_stale.assign(batch, 0);
    Workspace& ws = kv->ws;
    ws.prefill_rows = std::min(PREFILL_ROWS_MAX, (kv->max_len + 255) / 256 * 256);
    ws.r_max = std::max(ws.prefill_rows, batch * ANPD_ROWS);
    ws.n_max_out = (std::max(std::max(m->nqkv, 2 * c.d_ffn), std::max(c.d_model, c.vocab)) + 127) / 128 * 128;
    ws.splits_max = m->max_segs;
    ws.amax_blocks = (c.vocab + 1023) / 1024;
    const size_t R = ws.r_max, d = c.d_model, F = c.d_ffn, V = c.vocab, hd = c.head_dim, half = hd / 2;
    const size_t pool = (size_t)c.n_layers * kv->total_pages * c.n_kv_heads * KV_PAGE * hd * 2;
    const size_t n_part = (size_t)R * c.n_q_heads * kv->pages_per_seq;
    struct Item { void** ptr; size_t bytes; };
    std::vector<Item> items = {
        {(void**)&kv->kpool, pool}, {(void**)&kv->vpool, pool},
        {(void**)&kv->page_table, (size_t)kv->total_pages * 4},
        {(void**)&kv->rope_cos, (size_t)kv->max_len * half * 4}, {(void**)&kv->rope_sin, (size_t)kv->max_len * half * 4},
        {(void**)&kv->seq, sizeof(SeqState) * (size_t)batch}, {(void**)&kv->d_prompt, (size_t)kv->max_len * 4},
        {(void**)&kv->d_ctxs, sizeof(NgramDev) * (size_t)batch},
        {(void**)&ws.row_tok, R * 4}, {(void**)&ws.row_pos, R * 4}, {(void**)&ws.row_seq, R * 4}, {(void**)&ws.row_ok, R * 4},
        {(void**)&ws.row_slot, R * 4}, {(void**)&ws.row_hole_lo, R * 4}, {(void**)&ws.row_hole_hi, R * 4},
        {(void**)&ws.x, R * d * 4}, {(void**)&ws.h_hi, R * d * 2}, {(void**)&ws.h_lo, R * d * 2},
        {(void**)&ws.ao_hi, R * m->dq * 2}, {(void**)&ws.ao_lo, R * m->dq * 2},
        {(void**)&ws.act_hi, R * F * 2}, {(void**)&ws.act_lo, R * F * 2},
        // decode steps leave up to splits_max partial sums per output, prompt passes up to three (their cut along K)
        {(void**)&ws.part, std::max((size_t)ws.splits_max * batch * ANPD_ROWS, 3 * R) * ws.n_max_out * 4},
        {(void**)&ws.q_hi, R * m->dq * 2}, {(void**)&ws.q_lo, R * m->dq * 2},
        {(void**)&ws.attn_m, n_part * 4}, {(void**)&ws.attn_l, n_part * 4}, {(void**)&ws.attn_o, n_part * hd * 4},
        {(void**)&ws.logits, (size_t)batch * ANPD_ROWS * V * 4},
        {(void**)&ws.amax_val, R * ws.amax_blocks * 4}, {(void**)&ws.amax_idx, R * ws.amax_blocks * 4},
        {(void**)&ws.gemm_err, 256}, {(void**)&kv->loop_steps_left, 256},
        {(void**)&ws.img_h, act_img_bytes(c.d_model)}, {(void**)&ws.img_h2, act_img_bytes(c.d_model)},
        {(void**)&ws.img_ao, act_img_bytes(m->dq)}, {(void**)&ws.img_act, act_img_bytes(c.d_ffn)},
        {(void**)&ws.ss_a, (size_t)m->num_sms * ANPD_ROWS * 4}, {(void**)&ws.ss_b, (size_t)m->num_sms * ANPD_ROWS * 4},
        {(void**)&ws.amax_val_rr, (size_t)m->num_sms * ANPD_ROWS * 4}, {(void**)&ws.amax_idx_rr, (size_t)m->num_sms * ANPD_ROWS * 4},
    };
    ws.amax_nblk = ws.amax_blocks;
    size_t total = 0;
    for (const Item& it : items) total += up256(it.bytes);
    kv->slab_bytes = total;
    if (cudaMalloc(&kv->slab, total) != cudaSuccess) { cudaGetLastError(); delete kv; return ANPD_ERR_OOM; }
    char* p = (char*)kv->slab;
    for (const Item& it : items) { *it.ptr = p; p += up256(it.bytes); }
    const size_t pinned_bytes = sizeof(SeqState) * (size_t)batch + 64 * sizeof(int) * (size_t)batch + 256;
    if (cudaMallocHost((void**)&kv->h_seq, pinned_bytes) != cudaSuccess) { cudaGetLastError(); cudaFree(kv->slab); delete kv; return ANPD_ERR_OOM; }
    kv->h_small = (int*)((char*)kv->h_seq + sizeof(SeqState) * (size_t)batch);

    // TMA views of the GEMM inputs: decode rows (batch * 8) and prefill rows, each padded to the MMA's N
    {
        const int mode_rows[2] = {batch * ANPD_ROWS, ws.prefill_rows};
        anpd_status rc = ANPD_OK;
        for (int md = 0; md < 2 && rc == ANPD_OK; ++md) {
            const int rows = mode_rows[md], nb = md == 0 ? (rows + 15) / 16 * 16 : 128;
            ws.nb[md] = nb;
            struct { CUtensorMap* maps; const bf16* hi; const bf16* lo; int K; } bufs[3] = {
                {ws.map_h[md], ws.h_hi, ws.h_lo, c.d_model}, {ws.map_ao[md], ws.ao_hi, ws.ao_lo, m->dq}, {ws.map_act[md], ws.act_hi, ws.act_lo, c.d_ffn}};
            for (auto& bdesc : bufs) {
                // rows beyond the tensor's extent are zero-filled by the copy engine
                if (rc == ANPD_OK) rc = make_tmap_bf16(&bdesc.maps[0], bdesc.hi, rows, bdesc.K, nb, false);
                if (rc == ANPD_OK) rc = make_tmap_bf16(&bdesc.maps[1], bdesc.lo, rows, bdesc.K, nb, false);
            }
        }
        if (rc != ANPD_OK) { cudaFreeHost(kv->h_seq); cudaFree(kv->slab); delete kv; return rc; }
    }

    // TMA views of the K and V pools for the tensor-core attention: every page of every layer and kv head is 128 rows of hd
    kv->attn_tc = (c.head_dim == 128) && std::getenv("ANPD_ATTN_MMA_SYNC") == nullptr;
    kv->attn_pf = std::getenv("ANPD_ATTN_PROMPT_TILE16") == nullptr;
    if (kv->attn_tc) {
        const long long pool_rows = (long long)c.n_layers * kv->total_pages * c.n_kv_heads * KV_PAGE;
        anpd_status rc = pool_rows < (1ll << 31) ? ANPD_OK : ANPD_ERR_CAPACITY;
        if (rc == ANPD_OK) rc = make_tmap_bf16(&kv->map_k, kv->kpool, (int)pool_rows, c.head_dim, KV_PAGE, true);
        if (rc == ANPD_OK) rc = make_tmap_bf16(&kv->map_v, kv->vpool, (int)pool_rows, c.head_dim, KV_PAGE, true);
        if (rc == ANPD_OK) rc = make_tmap_bf16(&ws.map_q[0], ws.q_hi, ws.r_max, m->dq, 128, false);
        if (rc == ANPD_OK) rc = make_tmap_bf16(&ws.map_q[1], ws.q_lo, ws.r_max, m->dq, 128, false);
        if (rc != ANPD_OK) { cudaFreeHost(kv->h_seq); cudaFree(kv->slab); delete kv; return rc; }
    }

    ws.amax_val_use = ws.amax_val;
    ws.amax_idx_use = ws.amax_idx;
    {
        const anpd_status rc = step_kernel_setup(m, kv);
        if (rc != ANPD_OK) { cudaFree(kv->step_slab); cudaFreeHost(kv->h_seq); cudaFree(kv->slab); delete kv; return rc; }
    }

    // page table: identity, or a fixed permutation of the physical pages
    std::vector<int> pt(kv->total_pages);
    for (int i = 0; i < kv->total_pages; ++i) pt[i] = i;
    if (shuffle_pages) {
        uint64_t s = 0x9E3779B97F4A7C15ull;
        for (int i = kv->total_pages - 1; i > 0; --i) {
            s = s * 6364136223846793005ull + 1442695040888963407ull;
            std::swap(pt[i], pt[(int)((s >> 33) % (uint64_t)(i + 1))]);
        }
    }
    // rotary tables in double, rounded once to fp32: angle = pos * theta^(-2i/hd)
    std::vector<float> hc((size_t)kv->max_len * half), hs((size_t)kv->max_len * half);
    for (size_t i = 0; i < half; ++i) {
        const double inv = std::pow((double)c.rope_theta, -2.0 * (double)i / (double)hd);
        for (int pos = 0; pos < kv->max_len; ++pos) {
            hc[(size_t)pos * half + i] = (float)std::cos(pos * inv);
            hs[(size_t)pos * half + i] = (float)std::sin(pos * inv);
        }
    }
    cudaStream_t st = m->stream;
    bool ok = cudaMemsetAsync(kv->slab, 0, total, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(kv->page_table, pt.data(), pt.size() * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(kv->rope_cos, hc.data(), hc.size() * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(kv->rope_sin, hs.data(), hs.size() * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    std::memset(kv->h_seq, 0, sizeof(SeqState) * (size_t)batch);
    for (int b = 0; b < batch; ++b) { kv->h_seq[b].active = 1; kv->h_seq[b].stop_at = 0x7fffffff; }
    ok = ok && cudaMemcpyAsync(kv->seq, kv->h_seq, sizeof(SeqState) * (size_t)batch, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(st) == cudaSuccess;
    if (!ok) {
        anpd_note_cuda_error(cudaGetLastError(), __FILE__, __LINE__);
        cudaFree(kv->step_slab); cudaFreeHost(kv->h_seq); cudaFree(kv->slab); delete kv;
        return ANPD_ERR_CUDA;
    }
    *out = kv;
    return ANPD_OK;
}

anpd_status anpd_kv_destroy(anpd_kv* kv) {
    if (!kv) return ANPD_ERR_ARG;
    cudaStreamSynchronize(kv->m->stream);
    step_kernel_trace_dump(kv);
    for (auto& g : kv->graphs) cudaGraphExecDestroy(g.second.exec);
    for (auto& g : kv->loop_graphs) cudaGraphExecDestroy(g.second.exec);
    if (kv->side_stream) { cudaStreamSynchronize(kv->side_stream); cudaEventDestroy(kv->ev_fork); cudaEventDestroy(kv->ev_join); cudaStreamDestroy(kv->side_stream); }
    cudaFreeHost(kv->h_seq);
    cudaFree(kv->step_slab);
    cudaFree(kv->slab);
    delete kv;
    return ANPD_OK;
}

anpd_status anpd_kv_len(anpd_kv* kv, int seq, int* len) {
    if (!kv || !len || seq < 0 || seq >= kv->batch) return ANPD_ERR_ARG;
    *len = kv->h_kv_len[seq];
    return ANPD_OK;
}

anpd_status anpd_kv_truncate(anpd_kv* kv, int seq, int len) {
    if (!kv || seq < 0 || seq >= kv->batch || len < 0) return ANPD_ERR_ARG;
    if (len > kv->h_kv_len[seq]) return ANPD_ERR_RANGE;
    LAUNCH(&kv->m->prof, kv->m->stream, KC_OTHER, 0, (set_int_kernel<<<1, 1, 0, kv->m->stream>>>(&kv->seq[seq].kv_len, len)));
    CUDA_TRY(cudaGetLastError());
    kv->h_kv_len[seq] = len;
    kv->h_len_stale[seq] = 0;
    return ANPD_OK;
}

// Puts every sequence back to the empty state (device and host mirror).
static anpd_status kv_reset(anpd_kv* kv, const int* stop_at) {
    for (int b = 0; b < kv->batch; ++b) {
        std::memset(&kv->h_seq[b], 0, sizeof(SeqState));
        kv->h_seq[b].active = 1;
        kv->h_seq[b].stop_at = stop_at ? stop_at[b] : 0x7fffffff;
        kv->h_kv_len[b] = 0;
        kv->h_len_stale[b] = 0;
    }
    CUDA_TRY(cudaMemcpyAsync(kv->seq, kv->h_seq, sizeof(SeqState) * (size_t)kv->batch, cudaMemcpyHostToDevice, kv->m->stream));
    CUDA_TRY(cudaStreamSynchronize(kv->m->stream));
    return ANPD_OK;
}

// ---------------------------------------------------------------------------------------------
// prefill
// ---------------------------------------------------------------------------------------------
static anpd_status prefill_enqueue(anpd_model* m, anpd_kv* kv, int seq, const int32_t* prompt, int prompt_len,
                                   const NgramDev* d_ctxs) {
    CUDA_TRY(cudaMemcpyAsync(kv->d_prompt, prompt, sizeof(int) * (size_t)prompt_len, cudaMemcpyDefault, m->stream));
    const int pass_rows = kv->ws.prefill_rows;
    for (int start = 0; start < prompt_len; start += pass_rows) {
        const int n = std::min(pass_rows, prompt_len - start);
        const int rows = (n + ANPD_ROWS - 1) / ANPD_ROWS * ANPD_ROWS;
        const bool last = start + n >= prompt_len;
        // the row plan also covers the padding up to a multiple of 64 rows: the prompt attention takes up to 64 rows per item
        ANPD_TRY(plan_prefill_enqueue(m, kv, seq, start, prompt_len, std::min((rows + 63) / 64 * 64, kv->ws.r_max)));
        const int last_row = prompt_len - 1 - start;
        ANPD_TRY(forward_enqueue(m, kv, rows, std::min(start + rows - 1, kv->max_len - 1), last, false, last_row));
        // the LM head of a prompt pass runs on the last token's group of 8 rows, moved to rows 0-7
        if (last) ANPD_TRY(accept_enqueue(m, kv, ACCEPT_PREFILL, d_ctxs, seq, rows == kv->batch * ANPD_ROWS ? last_row : last_row % ANPD_ROWS, prompt_len));
    }
    return ANPD_OK;
}

static anpd_status read_seqs(anpd_kv* kv) {
    int* h_err = kv->h_small + 48 * kv->batch;
    CUDA_TRY(cudaMemcpyAsync(kv->h_seq, kv->seq, sizeof(SeqState) * (size_t)kv->batch, cudaMemcpyDeviceToHost, kv->m->stream));
    CUDA_TRY(cudaMemcpyAsync(h_err, kv->ws.gemm_err, sizeof(int), cudaMemcpyDeviceToHost, kv->m->stream));
    CUDA_TRY(cudaStreamSynchronize(kv->m->stream));
    for (int b = 0; b < kv->batch; ++b) { kv->h_kv_len[b] = kv->h_seq[b].kv_len; kv->h_len_stale[b] = 0; }
    if (*h_err != 0) {
        std::snprintf(g_last_error, sizeof(g_last_error), "a kernel gave up waiting on a barrier (code %d: 201 GEMM, 202 attention, 204 step kernel)", *h_err);
        return ANPD_ERR_CUDA;
    }
    return ANPD_OK;
}

static anpd_status seq_error_status(const SeqState& s) {
    if (s.error == 0) return ANPD_OK;
    if (s.error == 101) return ANPD_ERR_RANGE;
    if (s.error == 102 || s.error == 103) return ANPD_ERR_CAPACITY;
    return ANPD_ERR_CUDA;
}

anpd_status anpd_prefill(anpd_model* m, anpd_kv* kv, int seq, const int32_t* prompt, int prompt_len, int32_t* first_tok) {
    if (!m || !kv || !prompt || !first_tok || kv->m != m || seq < 0 || seq >= kv->batch || prompt_len < 1) return ANPD_ERR_ARG;
    ANPD_TRY(check_device(m));
    if (kv->h_kv_len[seq] != 0) return ANPD_ERR_STATE;
    if (prompt_len + ANPD_ROWS > kv->max_len) return ANPD_ERR_CAPACITY;
    for (int i = 0; i < prompt_len; ++i) if (prompt[i] < 0 || prompt[i] >= m->cfg.vocab) return ANPD_ERR_RANGE;
    LAUNCH(&m->prof, m->stream, KC_OTHER, 0, (seq_restart_kernel<<<1, 1, 0, m->stream>>>(&kv->seq[seq])));
    CUDA_TRY(cudaGetLastError());
    ANPD_TRY(prefill_enqueue(m, kv, seq, prompt, prompt_len, nullptr));
    ANPD_TRY(read_seqs(kv));
    ANPD_TRY(seq_error_status(kv->h_seq[seq]));
    *first_tok = kv->h_seq[seq].next_tok;
    return ANPD_OK;
}

// ---------------------------------------------------------------------------------------------
// verify
// ---------------------------------------------------------------------------------------------
anpd_status anpd_verify_stage(anpd_model* m, anpd_kv* kv, const int32_t* last_tok, const int32_t* drafts, const int* draft_len) {
    if (!m || !kv || kv->m != m || !last_tok || !draft_len) return ANPD_ERR_ARG;
    const int B = kv->batch;
    for (int b = 0; b < B; ++b) {
        if (draft_len[b] < 0 || draft_len[b] > ANPD_K_MAX) return ANPD_ERR_RANGE;
        if (draft_len[b] > 0 && !drafts) return ANPD_ERR_ARG;
        if (last_tok[b] < 0 || last_tok[b] >= m->cfg.vocab) return ANPD_ERR_RANGE;
        for (int i = 0; i < draft_len[b]; ++i)
            if (drafts[b * ANPD_K_MAX + i] < 0 || drafts[b * ANPD_K_MAX + i] >= m->cfg.vocab) return ANPD_ERR_RANGE;
    }
    // last_tok, draft_len and draft[] are adjacent in SeqState: one strided copy fills them
    const int W = 2 + ANPD_K_MAX + 1;
    CUDA_TRY(cudaStreamSynchronize(m->stream));          // the staging buffer may still be in use
    int* stage = kv->h_small;
    for (int b = 0; b < B; ++b) {
        stage[b * W + 0] = last_tok[b];
        stage[b * W + 1] = draft_len[b];
        for (int i = 0; i <= ANPD_K_MAX; ++i) stage[b * W + 2 + i] = (i < draft_len[b]) ? drafts[b * ANPD_K_MAX + i] : 0;
    }
    CUDA_TRY(cudaMemcpy2DAsync(&kv->seq[0].last_tok, sizeof(SeqState), stage, W * sizeof(int), W * sizeof(int), B,
                               cudaMemcpyHostToDevice, m->stream));
    kv->staged = true;
    return ANPD_OK;
}

// One draft-and-verify step for every sequence of the kv handle, enqueued on the model's stream.
// K > 0: fold the last step's tokens into the n-gram tables and draft K tokens; K == 0: plain greedy
// (the confirmed token alone); K < 0: the step's inputs were staged by the host.  Then the forward over
// the batch * 8 rows, argmax / accept and, in COMMIT mode, the KV commit and token-buffer append.
// Steps of one shape are captured once into a CUDA graph and replayed.
static anpd_status step_enqueue(anpd_model* m, anpd_kv* kv, int mode, bool want_logits, const NgramDev* d_ctxs, int K, int max_pos, bool two) {
    cudaStream_t st = m->stream;
    // Two candidates per step (the Conclusion's outlook on verifying several candidates at once): the first keeps up to 4
    // draft tokens, the alternative up to 3, so that both fit the step's 7 draft rows.
    // (`two`; a host-staged step, K < 0, brings both candidates itself.)
    if (K > 0) ANPD_TRY(ngram_enqueue_step(d_ctxs, kv->seq, kv->batch, two ? std::min(K, 4) : K, st, &m->prof, two ? std::min(K, 3) : 0));
    else if (K == 0) { LAUNCH(&m->prof, st, KC_OTHER, 0, (launch_k(greedy_stage_kernel, kv->batch, 1, 0, st, kv->seq))); }
    ANPD_TRY(plan_decode_enqueue(m, kv, two));
    ANPD_TRY(forward_enqueue(m, kv, kv->batch * ANPD_ROWS, max_pos, true, want_logits, 0, two));
    ANPD_TRY(accept_enqueue(m, kv, mode, d_ctxs, 0, 0, 0, two));
    return ANPD_OK;
}

// The whole decoding loop of Algorithm 1 as ONE graph launch: a conditional WHILE node whose body is the step (update +
// draft, row plan, forward, accept / commit) followed by a kernel that decides whether another step runs.  The host neither
// launches nor synchronises per step.  The body's attention grid is sized for the longest context the run can reach
// (`max_pos_bound`); pages beyond a sequence's current length are skipped inside the kernels.  Returns ANPD_ERR_STATE if
// the loop cannot be built on this stream / driver (the caller then steps from the host).
static anpd_status decode_loop_enqueue(anpd_model* m, anpd_kv* kv, const NgramDev* d_ctxs, int K, int max_pos_bound, int max_steps) {
    if (!kv->use_graphs || m->prof.on || !kv->loop_ok) return ANPD_ERR_STATE;
    cudaStream_t st = m->stream;
    const uint64_t key = (uint64_t)(max_pos_bound / KV_PAGE) | ((uint64_t)(K + 1) << 16) | ((uint64_t)(d_ctxs ? 1 : 0) << 29) |
                         ((uint64_t)(kv->candidates == 2 ? 1 : 0) << 30);
    auto it = kv->loop_graphs.find(key);
    if (it == kv->loop_graphs.end()) {
        if (!kv->warm) {                                // one eager step first: function attributes, lazy module loading
            kv->warm = true;
            return ANPD_ERR_STATE;
        }
        cudaGraph_t graph = nullptr;
        cudaGraphExec_t exec = nullptr;
        bool ok = cudaGraphCreate(&graph, 0) == cudaSuccess;
        cudaGraphConditionalHandle handle = 0;
        ok = ok && cudaGraphConditionalHandleCreate(&handle, graph, 1, cudaGraphCondAssignDefault) == cudaSuccess;
        cudaGraphNodeParams np = {};
        np.type = cudaGraphNodeTypeConditional;
        np.conditional.handle = handle;
        np.conditional.type = cudaGraphCondTypeWhile;
        np.conditional.size = 1;
        cudaGraphNode_t node = nullptr;
        ok = ok && cudaGraphAddNode(&node, graph, nullptr, 0, &np) == cudaSuccess;
        int launches = 0;
        if (ok) {
            cudaGraph_t body = np.conditional.phGraph_out[0];
            const long long before = g_launch_count.load();
            ok = cudaStreamBeginCaptureToGraph(st, body, nullptr, nullptr, 0, cudaStreamCaptureModeThreadLocal) == cudaSuccess;
            if (ok) {
                anpd_status rc = step_enqueue(m, kv, ACCEPT_COMMIT, false, d_ctxs, K, max_pos_bound, K > 0 && kv->candidates == 2);
                if (rc == ANPD_OK) {
                    LAUNCH(&m->prof, st, KC_OTHER, 0,
                           (launch_k(loop_condition_kernel, 1, 32, 0, st, kv->seq, kv->batch, kv->ws.gemm_err, kv->loop_steps_left, handle)));
                    if (cudaGetLastError() != cudaSuccess) rc = ANPD_ERR_CUDA;
                }
                cudaGraph_t captured = nullptr;
                const cudaError_t ce = cudaStreamEndCapture(st, &captured);
                ok = rc == ANPD_OK && ce == cudaSuccess;
            }
            launches = (int)(g_launch_count.load() - before);
            g_launch_count.fetch_sub(launches);         // capturing runs nothing
        }
        ok = ok && cudaGraphInstantiate(&exec, graph, 0) == cudaSuccess;
        if (graph) cudaGraphDestroy(graph);
        if (!ok) {
            cudaGetLastError();
            if (exec) cudaGraphExecDestroy(exec);
            kv->loop_ok = false;                        // step from the host for good
            return ANPD_ERR_STATE;
        }
        it = kv->loop_graphs.emplace(key, anpd_kv::StepGraph{exec, launches}).first;
    }
    CUDA_TRY(cudaMemcpyAsync(kv->loop_steps_left, &max_steps, sizeof(int), cudaMemcpyHostToDevice, st));
    CUDA_TRY(cudaGraphLaunch(it->second.exec, st));
    std::fill(kv->h_len_stale.begin(), kv->h_len_stale.end(), 1);
    kv->loop_launches_per_step = it->second.launches;
    return ANPD_OK;
}

static anpd_status verify_enqueue_mode(anpd_model* m, anpd_kv* kv, int mode, bool want_logits, const NgramDev* d_ctxs, int K = -1, bool two = false) {
    ANPD_TRY(check_device(m));
    int max_pos = 0;
    for (int b = 0; b < kv->batch; ++b) {
        // the attention grid is sized from the host's copy of the lengths: it must not be behind the device
        if (kv->h_len_stale[b]) return ANPD_ERR_STATE;
        if (kv->h_kv_len[b] + ANPD_ROWS > kv->max_len) return ANPD_ERR_CAPACITY;
        max_pos = std::max(max_pos, kv->h_kv_len[b] + ANPD_ROWS - 1);
    }
    cudaStream_t st = m->stream;
    auto enqueue = [&]() -> anpd_status { return step_enqueue(m, kv, mode, want_logits, d_ctxs, K, max_pos, two); };
    if (m->prof.on || !kv->use_graphs || !kv->warm) {
        kv->warm = true;
        NoPdlScope no_overlap(m->prof.on);            // per-launch timing needs kernels that do not overlap
        const anpd_status rc = enqueue();
        if (rc == ANPD_OK && mode == ACCEPT_COMMIT) std::fill(kv->h_len_stale.begin(), kv->h_len_stale.end(), 1);
        return rc;
    }
    const uint64_t key = (uint64_t)(max_pos / KV_PAGE) | ((uint64_t)(K + 1) << 16) | ((uint64_t)mode << 24) |
                         ((uint64_t)(want_logits ? 1 : 0) << 28) | ((uint64_t)(d_ctxs ? 1 : 0) << 29) | ((uint64_t)(two ? 1 : 0) << 30);
    auto it = kv->graphs.find(key);
    if (it == kv->graphs.end()) {
        const long long before = g_launch_count.load();
        cudaGraph_t graph = nullptr;
        if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
            cudaGetLastError();
            kv->use_graphs = false;
            { const anpd_status r2 = enqueue(); if (r2 == ANPD_OK && mode == ACCEPT_COMMIT) std::fill(kv->h_len_stale.begin(), kv->h_len_stale.end(), 1); return r2; }
        }
        const anpd_status rc = enqueue();
        const cudaError_t ce = cudaStreamEndCapture(st, &graph);
        const int launches = (int)(g_launch_count.load() - before);
        g_launch_count.fetch_sub(launches);           // capturing runs nothing
        anpd_kv::StepGraph sg{nullptr, launches};
        if (rc != ANPD_OK || ce != cudaSuccess || !graph || cudaGraphInstantiate(&sg.exec, graph, 0) != cudaSuccess) {
            cudaGetLastError();
            if (graph) cudaGraphDestroy(graph);
            kv->use_graphs = false;                   // fall back to plain launches for good
            { const anpd_status r2 = enqueue(); if (r2 == ANPD_OK && mode == ACCEPT_COMMIT) std::fill(kv->h_len_stale.begin(), kv->h_len_stale.end(), 1); return r2; }
        }
        cudaGraphDestroy(graph);
        it = kv->graphs.emplace(key, sg).first;
    }
    CUDA_TRY(cudaGraphLaunch(it->second.exec, st));
    g_launch_count += it->second.launches;
    if (mode == ACCEPT_COMMIT) std::fill(kv->h_len_stale.begin(), kv->h_len_stale.end(), 1);
    return ANPD_OK;
}

anpd_status anpd_kv_set_candidates(anpd_kv* kv, int candidates) {
    if (!kv) return ANPD_ERR_ARG;
    if (candidates != 1 && candidates != 2) return ANPD_ERR_RANGE;
    kv->candidates = candidates;
    return ANPD_OK;
}

anpd_status anpd_verify_enqueue(anpd_model* m, anpd_kv* kv) {
    if (!m || !kv || kv->m != m) return ANPD_ERR_ARG;
    if (!kv->staged) return ANPD_ERR_STATE;
    return verify_enqueue_mode(m, kv, ACCEPT_COMMIT, false, nullptr);
}

anpd_status anpd_verify_result(anpd_model* m, anpd_kv* kv, int* accepted_len, int32_t* next_tok) {
    if (!m || !kv || kv->m != m || !accepted_len || !next_tok) return ANPD_ERR_ARG;
    ANPD_TRY(read_seqs(kv));
    for (int b = 0; b < kv->batch; ++b) ANPD_TRY(seq_error_status(kv->h_seq[b]));
    for (int b = 0; b < kv->batch; ++b) { accepted_len[b] = kv->h_seq[b].accepted_len; next_tok[b] = kv->h_seq[b].next_tok; }
    return ANPD_OK;
}

anpd_status anpd_verify_batch(anpd_model* m, anpd_kv* kv, const int32_t* last_tok, const int32_t* drafts,
                              const int* draft_len, int* accepted_len, int32_t* next_tok) {
    if (!accepted_len || !next_tok) return ANPD_ERR_ARG;
    ANPD_TRY(anpd_verify_stage(m, kv, last_tok, drafts, draft_len));
    ANPD_TRY(anpd_verify_enqueue(m, kv));
    return anpd_verify_result(m, kv, accepted_len, next_tok);
}

anpd_status anpd_verify(anpd_model* m, anpd_kv* kv, int32_t last_tok, const int32_t* draft, int draft_len,
                        int* accepted_len, int32_t* next_tok) {
    if (!kv || kv->batch != 1) return ANPD_ERR_ARG;
    int32_t padded[ANPD_K_MAX] = {0};
    if (draft_len < 0 || draft_len > ANPD_K_MAX) return ANPD_ERR_RANGE;
    if (draft_len > 0 && !draft) return ANPD_ERR_ARG;
    for (int i = 0; i < draft_len; ++i) padded[i] = draft[i];
    return anpd_verify_batch(m, kv, &last_tok, padded, &draft_len, accepted_len, next_tok);
}

anpd_status anpd_verify_logits(anpd_model* m, anpd_kv* kv, int32_t last_tok, const int32_t* draft, int draft_len,
                               float* logits_host) {
    if (!kv || kv->batch != 1 || !logits_host) return ANPD_ERR_ARG;
    int32_t padded[ANPD_K_MAX] = {0};
    if (draft_len < 0 || draft_len > ANPD_K_MAX) return ANPD_ERR_RANGE;
    if (draft_len > 0 && !draft) return ANPD_ERR_ARG;
    for (int i = 0; i < draft_len; ++i) padded[i] = draft[i];
    ANPD_TRY(anpd_verify_stage(m, kv, &last_tok, padded, &draft_len));
    ANPD_TRY(verify_enqueue_mode(m, kv, ACCEPT_PEEK, true, nullptr));
    CUDA_TRY(cudaMemcpyAsync(logits_host, kv->ws.logits, sizeof(float) * (size_t)(draft_len + 1) * m->cfg.vocab,
                             cudaMemcpyDeviceToHost, m->stream));
    ANPD_TRY(read_seqs(kv));
    return seq_error_status(kv->h_seq[0]);
}

anpd_status anpd_verify_two_candidates(anpd_model* m, anpd_kv* kv, int32_t last_tok, const int32_t* draft_a, int len_a,
                                       const int32_t* draft_b, int len_b, int* accepted_len, int32_t* next_tok, int* chosen,
                                       float* logits_host) {
    if (!m || !kv || kv->m != m || kv->batch != 1 || !accepted_len || !next_tok || !chosen || !draft_a || !draft_b) return ANPD_ERR_ARG;
    if (len_a < 1 || len_b < 1 || len_a + len_b > ANPD_K_MAX) return ANPD_ERR_RANGE;
    for (int i = 0; i < len_b; ++i)
        if (draft_b[i] < 0 || draft_b[i] >= m->cfg.vocab) return ANPD_ERR_RANGE;
    int32_t padded[ANPD_K_MAX] = {0};
    for (int i = 0; i < len_a; ++i) padded[i] = draft_a[i];
    ANPD_TRY(anpd_verify_stage(m, kv, &last_tok, padded, &len_a));
    // draft2_len and draft2[] are adjacent in SeqState too
    int* stage = kv->h_small + (2 + ANPD_K_MAX + 1);
    stage[0] = len_b;
    for (int i = 0; i <= ANPD_K_MAX; ++i) stage[1 + i] = (i < len_b) ? draft_b[i] : 0;
    CUDA_TRY(cudaMemcpyAsync(&kv->seq[0].draft2_len, stage, (2 + ANPD_K_MAX) * sizeof(int), cudaMemcpyHostToDevice, m->stream));
    ANPD_TRY(verify_enqueue_mode(m, kv, ACCEPT_COMMIT, logits_host != nullptr, nullptr, -1, true));
    if (logits_host)
        CUDA_TRY(cudaMemcpyAsync(logits_host, kv->ws.logits, sizeof(float) * (size_t)(len_a + len_b + 1) * m->cfg.vocab,
                                 cudaMemcpyDeviceToHost, m->stream));
    ANPD_TRY(read_seqs(kv));
    ANPD_TRY(seq_error_status(kv->h_seq[0]));
    *accepted_len = kv->h_seq[0].accepted_len;
    *next_tok = kv->h_seq[0].next_tok;
    *chosen = kv->h_seq[0].move_n > 0 ? 1 : 0;
    return ANPD_OK;
}

// ---------------------------------------------------------------------------------------------
// Algorithm 1
// ---------------------------------------------------------------------------------------------
static anpd_status generate_core(anpd_model* m, anpd_kv* kv, anpd_ngram* const* ctxs, const int32_t* prompts,
                                 int prompt_len, int max_new, int K, int32_t* out, anpd_stats* stats, bool on_device) {
    if (!m || !kv || kv->m != m || !ctxs || !prompts || !out || prompt_len < 1 || max_new < 1) return ANPD_ERR_ARG;
    if (K < 0 || K > ANPD_K_MAX) return ANPD_ERR_RANGE;
    ANPD_TRY(check_device(m));
    const int B = kv->batch;
    cudaStream_t st = m->stream;
    for (int b = 0; b < B; ++b) {
        if (!ctxs[b] || ctxs[b]->stream != st) return ANPD_ERR_ARG;
        if (prompt_len + max_new + 1 + ANPD_ROWS > ctxs[b]->h.max_ctx) return ANPD_ERR_CAPACITY;
    }
    if (prompt_len + max_new + 2 * ANPD_ROWS > kv->max_len) return ANPD_ERR_CAPACITY;
    if (!on_device)
        for (size_t i = 0; i < (size_t)B * prompt_len; ++i) if (prompts[i] < 0 || prompts[i] >= m->cfg.vocab) return ANPD_ERR_RANGE;

    // Algorithm 1 tests length(O) < M at the top of the loop, where O receives the token confirmed by
    // the previous step; the context holds that pending token too, hence the + 1
    std::vector<int> stop(B, prompt_len + max_new + 1);
    ANPD_TRY(kv_reset(kv, stop.data()));
    std::vector<NgramDev> hd(B);
    for (int b = 0; b < B; ++b) {
        ANPD_TRY(anpd_ngram_reset(ctxs[b]));
        hd[b] = ctxs[b]->h;
    }
    CUDA_TRY(cudaMemcpyAsync(kv->d_ctxs, hd.data(), sizeof(NgramDev) * (size_t)B, cudaMemcpyHostToDevice, st));
    CUDA_TRY(cudaStreamSynchronize(st));

    cudaEvent_t e0, e1, e2;
    CUDA_TRY(cudaEventCreate(&e0)); CUDA_TRY(cudaEventCreate(&e1)); CUDA_TRY(cudaEventCreate(&e2));
    anpd_status rc = ANPD_OK;
    auto body = [&]() -> anpd_status {
        CUDA_TRY(cudaEventRecord(e0, st));
        // Initialize: the prompt's statistics (skipped for plain greedy, which never queries them)
        for (int b = 0; b < B; ++b) {
            anpd_ngram* c = ctxs[b];
            CUDA_TRY(cudaMemcpyAsync(c->h.tokens, prompts + (size_t)b * prompt_len, sizeof(int) * (size_t)prompt_len,
                                     cudaMemcpyDefault, st));
            kv->h_small[2 * b] = prompt_len; kv->h_small[2 * b + 1] = (K > 0) ? prompt_len : 0;
            CUDA_TRY(cudaMemcpyAsync(c->h.state, kv->h_small + 2 * b, 2 * sizeof(int), cudaMemcpyHostToDevice, st));
        }
        // the tables are not needed before the first draft: their kernels run beside the prompt passes, on the side stream
        if (K > 0 && kv->side_stream) {
            CUDA_TRY(cudaEventRecord(kv->ev_fork, st));
            CUDA_TRY(cudaStreamWaitEvent(kv->side_stream, kv->ev_fork, 0));
            for (int b = 0; b < B; ++b) ANPD_TRY(ngram_enqueue_bulk(ctxs[b], 0, prompt_len, &m->prof, kv->side_stream));
            CUDA_TRY(cudaEventRecord(kv->ev_join, kv->side_stream));
        } else if (K > 0) {
            for (int b = 0; b < B; ++b) ANPD_TRY(ngram_enqueue_bulk(ctxs[b], 0, prompt_len, &m->prof));
        }
        // LLM(prompt): the first token lands in the context as its first uncounted token
        for (int b = 0; b < B; ++b) ANPD_TRY(prefill_enqueue(m, kv, b, prompts + (size_t)b * prompt_len, prompt_len, kv->d_ctxs));
        if (K > 0 && kv->side_stream) CUDA_TRY(cudaStreamWaitEvent(st, kv->ev_join, 0));
        CUDA_TRY(cudaEventRecord(e1, st));
        ANPD_TRY(read_seqs(kv));
        for (int b = 0; b < B; ++b) ANPD_TRY(seq_error_status(kv->h_seq[b]));
        bool any_active = true;
        while (any_active) {
            // the device-resident loop runs every remaining step in one launch; where it is not available (first step of a
            // handle, legacy stream, profiling, a driver that refuses the graph) the host steps and reads the state back
            const int max_pos_bound = std::min(prompt_len + max_new + 2 * ANPD_ROWS, kv->max_len) - 1;
            const anpd_status lrc = decode_loop_enqueue(m, kv, kv->d_ctxs, K, max_pos_bound, max_new + 2);
            if (lrc == ANPD_OK) g_launch_count += 0;    // counted below from the steps the sequences report
            else if (lrc != ANPD_ERR_STATE) return lrc;
            else ANPD_TRY(verify_enqueue_mode(m, kv, ACCEPT_COMMIT, false, kv->d_ctxs, K, K > 0 && kv->candidates == 2));
            int steps_before = 0;
            for (int b = 0; b < B; ++b) steps_before = std::max(steps_before, kv->h_seq[b].steps);
            ANPD_TRY(read_seqs(kv));
            any_active = false;
            int steps_after = 0;
            for (int b = 0; b < B; ++b) {
                ANPD_TRY(seq_error_status(kv->h_seq[b]));
                any_active = any_active || kv->h_seq[b].active;
                steps_after = std::max(steps_after, kv->h_seq[b].steps);
            }
            if (lrc == ANPD_OK) g_launch_count += (long long)kv->loop_launches_per_step * std::max(steps_after - steps_before, 1);
        }
        CUDA_TRY(cudaEventRecord(e2, st));
        CUDA_TRY(cudaEventSynchronize(e2));
        return ANPD_OK;
    };
    rc = body();
    if (rc == ANPD_OK) {
        float ms_p = 0, ms_d = 0;
        cudaEventElapsedTime(&ms_p, e0, e1);
        cudaEventElapsedTime(&ms_d, e1, e2);
        for (int b = 0; b < B && rc == ANPD_OK; ++b) {
            if (cudaMemcpy(out + (size_t)b * max_new, ctxs[b]->h.tokens + prompt_len, sizeof(int) * (size_t)max_new,
                           cudaMemcpyDefault) != cudaSuccess) { anpd_note_cuda_error(cudaGetLastError(), __FILE__, __LINE__); rc = ANPD_ERR_CUDA; break; }
            int nst[2] = {0, 0};
            if (cudaMemcpy(nst, ctxs[b]->h.state, 2 * sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) { rc = ANPD_ERR_CUDA; break; }
            const int nt = nst[0];
            ctxs[b]->n_tokens = nt;
            ctxs[b]->n_folded = (K > 0) ? nst[1] : 0;
            if (stats) {
                const SeqState& s = kv->h_seq[b];
                anpd_stats& o = stats[b];
                o.steps = s.steps; o.drafted = s.drafted; o.accepted = s.accepted; o.generated = nt - prompt_len - 1;
                for (int i = 0; i < 8; ++i) o.hist_accepted[i] = s.hist[i];
                o.alt_wins = s.alt_wins; o.reserved = 0;
                o.ms_prefill = ms_p; o.ms_decode = ms_d;
                const double mean_kv = prompt_len + 0.5 * (nt - prompt_len - 1);
                const anpd_model_config& c = m->cfg;
                o.bytes_per_step = m->streamed_bytes + B * mean_kv * (2.0 * c.n_layers * c.n_kv_heads * c.head_dim * 2.0);
            }
        }
    }
    cudaEventDestroy(e0); cudaEventDestroy(e1); cudaEventDestroy(e2);
    return rc;
}

anpd_status anpd_generate_batch(anpd_model* m, anpd_kv* kv, anpd_ngram* const* ctxs, const int32_t* prompts,
                                int prompt_len, int max_new, int K, int32_t* out, anpd_stats* stats) {
    return generate_core(m, kv, ctxs, prompts, prompt_len, max_new, K, out, stats, false);
}

anpd_status anpd_generate(anpd_model* m, anpd_kv* kv, anpd_ngram* ctx, const int32_t* prompt, int prompt_len,
                          int max_new, int K, int32_t* out, int* n_out, anpd_stats* stats) {
    if (!kv || kv->batch != 1 || !n_out) return ANPD_ERR_ARG;
    anpd_ngram* arr[1] = {ctx};
    ANPD_TRY(generate_core(m, kv, arr, prompt, prompt_len, max_new, K, out, stats, false));
    *n_out = max_new;
    return ANPD_OK;
}

anpd_status anpd_generate_dev(anpd_model* m, anpd_kv* kv, anpd_ngram* ctx, const int32_t* prompt_dev, int prompt_len,
                              int max_new, int K, int32_t* out_dev, int* n_out, anpd_stats* stats) {
    if (!kv || kv->batch != 1 || !n_out) return ANPD_ERR_ARG;
    anpd_ngram* arr[1] = {ctx};
    ANPD_TRY(generate_core(m, kv, arr, prompt_dev, prompt_len, max_new, K, out_dev, stats, true));
    *n_out = max_new;
    return ANPD_OK;
}

// ---------------------------------------------------------------------------------------------
// GEMM test hook
// ---------------------------------------------------------------------------------------------
// The product through the row-range kernel of single-sequence steps (exactly 8 rows), plain epilogue.
static anpd_status debug_gemm_row_range(const uint16_t* w_bf16, int N, int K, const float* a, float* out) {
    int dev = 0, sms = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    RRPlan plan;
    rr_make_plan(&plan, N, K, sms);
    const size_t wb = up256(rr_storage_bytes(plan)), ib = up256(act_img_bytes(K)), sb = up256((size_t)N * K * 2),
                 ab = up256((size_t)ANPD_ROWS * K * 4), ob = up256((size_t)ANPD_ROWS * N * 4);
    char* slab = nullptr;
    if (cudaMalloc((void**)&slab, wb + ib + sb + ab + ob + 256) != cudaSuccess) { cudaGetLastError(); return ANPD_ERR_OOM; }
    unsigned char* dW = (unsigned char*)slab;
    unsigned char* dimg = dW + wb;
    void* dsrc = dimg + ib;
    float* da = (float*)((char*)dsrc + sb);
    float* dout = (float*)((char*)da + ab);
    int* derr = (int*)((char*)dout + ob);
    auto body = [&]() -> anpd_status {
        CUDA_TRY(cudaMemset(slab, 0, wb + ib));
        CUDA_TRY(cudaMemset(dout, 0, ob + 256));
        CUDA_TRY(cudaMemcpy(dsrc, w_bf16, (size_t)N * K * 2, cudaMemcpyHostToDevice));
        CUDA_TRY(cudaMemcpy(da, a, (size_t)ANPD_ROWS * K * 4, cudaMemcpyHostToDevice));
        ANPD_TRY(rr_retile_enqueue(plan, dsrc, false, N, 0, RR_MAP_IDENTITY, 0, 0, dW, 0));
        ANPD_TRY(rr_act_image_enqueue(da, K, dimg, 0));
        CUDA_TRY(cudaDeviceSynchronize());
        RREpiHost e;
        e.raw_out = dout;
        ANPD_TRY(rr_enqueue(RR_RAW, plan, dW, dimg, e, derr, 0, nullptr));
        CUDA_TRY(cudaDeviceSynchronize());
        int err = 0;
        CUDA_TRY(cudaMemcpy(&err, derr, 4, cudaMemcpyDeviceToHost));
        if (err) { std::snprintf(g_last_error, sizeof(g_last_error), "GEMM kernel gave up waiting (code %d)", err); return ANPD_ERR_CUDA; }
        CUDA_TRY(cudaMemcpy(out, dout, (size_t)ANPD_ROWS * N * 4, cudaMemcpyDeviceToHost));
        return ANPD_OK;
    };
    const anpd_status rc = body();
    cudaFree(slab);
    return rc;
}

anpd_status anpd_debug_gemm(const uint16_t* w_bf16, int N, int K, const float* a, int rows, float* out, int plain) {
    if (!w_bf16 || !a || !out || N < 1 || K < 8 || K % 8 || rows < 8 || rows % 8 || rows > 128) return ANPD_ERR_ARG;
    if (plain == 2 && rows != ANPD_ROWS) return ANPD_ERR_ARG;
    if (!have_device()) return ANPD_ERR_CUDA;
    if (plain == 2) return debug_gemm_row_range(w_bf16, N, K, a, out);
    int dev = 0, sms = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    GemmPlan plan;
    gemm_make_plan(&plan, N, K, sms);
    const int NB = (rows + 15) / 16 * 16;
    const int segs = plain ? 1 : plan.max_segs;
    std::vector<uint16_t> hi((size_t)rows * K), lo((size_t)rows * K);
    for (size_t i = 0; i < hi.size(); ++i) {
        hi[i] = f32_to_bf16_host(a[i]);
        uint32_t u = (uint32_t)hi[i] << 16;
        float h; std::memcpy(&h, &u, 4);
        lo[i] = f32_to_bf16_host(a[i] - h);
    }
    const size_t wb = up256(gemm_tiled_elems(plan) * 2), ab = up256((size_t)rows * K * 2), pb = up256((size_t)segs * rows * N * 4),
                 tb = up256((size_t)plan.m_tiles * 4), sb = up256((size_t)N * K * 2);
    char* slab = nullptr;
    if (cudaMalloc((void**)&slab, wb + 2 * ab + pb + tb + 256 + sb) != cudaSuccess) { cudaGetLastError(); return ANPD_ERR_OOM; }
    void* dsrc = slab + wb + 2 * ab + pb + tb + 256;
    bf16* dW = (bf16*)slab; bf16* dhi = (bf16*)(slab + wb); bf16* dlo = (bf16*)(slab + wb + ab);
    float* dpart = (float*)(slab + wb + 2 * ab);
    int* dfirst = (int*)(slab + wb + 2 * ab + pb);
    int* derr = (int*)(slab + wb + 2 * ab + pb + tb);
    plan.d_first_cta = dfirst;
    anpd_status rc = ANPD_OK;
    auto body = [&]() -> anpd_status {
        CUDA_TRY(cudaMemset(slab, 0, wb));
        CUDA_TRY(cudaMemset(slab + wb + 2 * ab, 0, pb + tb + 256));
        CUDA_TRY(cudaMemcpy(dsrc, w_bf16, (size_t)N * K * 2, cudaMemcpyHostToDevice));
        ANPD_TRY(gemm_retile_enqueue(plan, dsrc, false, N, 0, dW, 0));
        CUDA_TRY(cudaMemcpy(dhi, hi.data(), hi.size() * 2, cudaMemcpyHostToDevice));
        CUDA_TRY(cudaMemcpy(dlo, lo.data(), lo.size() * 2, cudaMemcpyHostToDevice));
        CUDA_TRY(cudaMemcpy(dfirst, plan.first_cta.data(), (size_t)plan.m_tiles * 4, cudaMemcpyHostToDevice));
        if (plain) {
            ANPD_TRY(gemm_plain_enqueue(plan, dW, dhi, dlo, rows, dpart, N, 0, nullptr));
        } else {
            CUtensorMap mh, ml;
            ANPD_TRY(make_tmap_bf16(&mh, dhi, rows, K, NB, false));
            ANPD_TRY(make_tmap_bf16(&ml, dlo, rows, K, NB, false));
            ANPD_TRY(gemm_tc_enqueue(plan, dW, mh, ml, rows, NB, dpart, (size_t)rows * N, N, derr, 0, nullptr));
        }
        CUDA_TRY(cudaDeviceSynchronize());
        int err = 0;
        CUDA_TRY(cudaMemcpy(&err, derr, 4, cudaMemcpyDeviceToHost));
        if (err) { std::snprintf(g_last_error, sizeof(g_last_error), "GEMM kernel gave up waiting (code %d)", err); return ANPD_ERR_CUDA; }
        std::vector<float> part((size_t)segs * rows * N);
        CUDA_TRY(cudaMemcpy(part.data(), dpart, part.size() * 4, cudaMemcpyDeviceToHost));
        for (int r = 0; r < rows; ++r)
            for (int n = 0; n < N; ++n) {
                const int ns = plain ? 1 : plan.seg_count[n >> 7];
                float acc = 0.0f;
                for (int sgm = 0; sgm < ns; ++sgm) acc += part[((size_t)sgm * rows + r) * N + n];
                out[(size_t)r * N + n] = acc;
            }
        return ANPD_OK;
    };
    rc = body();
    cudaFree(slab);
    return rc;
}

// ---------------------------------------------------------------------------------------------
// measurement
// ---------------------------------------------------------------------------------------------
anpd_status anpd_profile_enable(anpd_model* m, int on) {
    if (!m) return ANPD_ERR_ARG;
    CUDA_TRY(cudaStreamSynchronize(m->stream));
    m->prof.drain();
    m->prof.on = on != 0;
    return ANPD_OK;
}

anpd_status anpd_profile_read(anpd_model* m, anpd_profile* out, int reset) {
    if (!m || !out) return ANPD_ERR_ARG;
    CUDA_TRY(cudaStreamSynchronize(m->stream));
    m->prof.drain();
    out->ms_gemm = m->prof.ms[KC_GEMM]; out->n_gemm = m->prof.n[KC_GEMM];
    out->ms_attn = m->prof.ms[KC_ATTN]; out->n_attn = m->prof.n[KC_ATTN];
    out->ms_other = m->prof.ms[KC_OTHER]; out->n_other = m->prof.n[KC_OTHER];
    out->ms_ngram = m->prof.ms[KC_NGRAM]; out->n_ngram = m->prof.n[KC_NGRAM];
    out->gemm_bytes = m->prof.gemm_bytes;
    if (reset) m->prof.clear();
    return ANPD_OK;
}

}  // extern "C"
