// Internal declarations shared by the library's translation units (not part of the boundary).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <atomic>
#include <map>
#include <vector>

#include "anpd.h"

// ---------------------------------------------------------------------------------------------
// error handling
// ---------------------------------------------------------------------------------------------
void anpd_note_cuda_error(cudaError_t e, const char* file, int line);

#define CUDA_TRY(expr)                                            \
    do {                                                          \
        cudaError_t e__ = (expr);                                 \
        if (e__ != cudaSuccess) {                                 \
            anpd_note_cuda_error(e__, __FILE__, __LINE__);        \
            return ANPD_ERR_CUDA;                                 \
        }                                                         \
    } while (0)

#define ANPD_TRY(expr)                       \
    do {                                     \
        anpd_status s__ = (expr);            \
        if (s__ != ANPD_OK) return s__;      \
    } while (0)

// One-time per-device set-up inside a launch helper (function attributes are per device): true the first time it
// is called for the current device with this flag array, which the caller keeps as a function-local static.
inline bool first_call_on_device(bool (&done)[64]) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return true;
    if (done[dev]) return false;
    done[dev] = true;
    return true;
}

// ---------------------------------------------------------------------------------------------
// launch accounting + optional per-class timing
// ---------------------------------------------------------------------------------------------
enum KernelClass { KC_GEMM = 0, KC_ATTN = 1, KC_OTHER = 2, KC_NGRAM = 3, KC_COUNT = 4 };

struct Profiler {
    bool on = false;
    std::vector<cudaEvent_t> ev;      // pairs
    std::vector<int> cls;             // class per pair
    std::vector<double> bytes;        // bytes per pair (GEMM weight bytes)
    size_t used = 0;                  // pairs in use
    double ms[KC_COUNT] = {0, 0, 0, 0};
    int n[KC_COUNT] = {0, 0, 0, 0};
    double gemm_bytes = 0;
    void begin(cudaStream_t st, int c, double b);
    void end(cudaStream_t st);
    void drain();                     // synchronises the events and folds them into ms/n
    void clear();
    ~Profiler();
};

extern std::atomic<long long> g_launch_count;

// Wraps one kernel launch: counts it and, when profiling, brackets it with events.
#define LAUNCH(prof, stream, kclass, wbytes, ...)                      \
    do {                                                               \
        Profiler* p__ = (prof);                                        \
        if (p__ && p__->on) p__->begin((stream), (kclass), (wbytes));  \
        __VA_ARGS__;                                                   \
        ++g_launch_count;                                              \
        if (p__ && p__->on) p__->end((stream));                        \
    } while (0)

// ---------------------------------------------------------------------------------------------
// programmatic dependent launch
// Every kernel of a step is launched so that it may start while its predecessor is still running:
// it signals its own successor at once (pdl_trigger) and blocks in pdl_wait before it touches
// anything an earlier kernel produced (or overwrites anything an earlier kernel may still read).
// The weight-streaming GEMM uses the gap: its producer thread requests the first weight tiles before
// it waits, so HBM keeps streaming through the small kernels between two GEMMs.  A kernel launched
// without the attribute (or with ANPD_NO_PDL set) sees both calls as no-ops.
// g_use_pdl is fixed when the library is loaded; t_no_pdl switches the attribute off for the launches
// the calling thread makes while it is set (per-launch timing; a GEMM whose weights were written by
// the kernel just before it and must therefore not be requested ahead of the dependency wait).
// ---------------------------------------------------------------------------------------------
extern const bool g_use_pdl;
extern thread_local bool t_no_pdl;
struct NoPdlScope {
    bool saved;
    explicit NoPdlScope(bool off) : saved(t_no_pdl) { if (off) t_no_pdl = true; }
    ~NoPdlScope() { t_no_pdl = saved; }
};
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (g_use_pdl && !t_no_pdl) ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

// ---------------------------------------------------------------------------------------------
// per-sequence step state (device)
// ---------------------------------------------------------------------------------------------
struct SeqState {
    int kv_len;                    // P: positions held by the cache
    int last_tok;                  // confirmed token fed as row 0
    int draft_len;                 // k <= K
    int draft[ANPD_K_MAX + 1];
    int accepted_len;              // a
    int next_tok;                  // the model's token after the last accepted draft
    int pred[ANPD_ROWS];           // argmax per row
    int steps, drafted, accepted;  // counters of the decoding loop
    int hist[8];
    int active;                    // 0: the sequence idles (finished or out of room)
    int stop_at;                   // the loop retires the sequence once its context holds this many tokens
    int error;                     // sticky device-side error code
    // a second candidate of the step (two-candidate mode): its tokens, how often it won, and the cache rows the accept
    // step asks to be moved when it wins (its rows were written behind the first candidate's)
    int draft2_len;
    int draft2[ANPD_K_MAX + 1];
    int alt_wins;
    int move_from, move_to, move_n;
};

// ---------------------------------------------------------------------------------------------
// n-gram tables (device)
// ---------------------------------------------------------------------------------------------
// Both tables of a level identify a key by a position: ref = t + 1 where t is a position of the
// committed sequence at which the n-gram x[t-n+1..t] occurred (0 = empty slot).  The key's
// tokens are read from the token buffer, which never changes below n_tokens.
struct GramSlot {      // one record per distinct n-gram
    int ref;
    int count;         // occurrences
    int last;          // last position t
    int pad;
};
struct PrefSlot {      // one record per distinct (n-1)-gram context
    int ref;
    int pad;
    unsigned long long best;   // packed (count | last_pos | successor), larger is better
};

struct NgramDev {
    int* tokens;       // [max_ctx]
    int* state;        // [0] n_tokens, [1] first position not yet folded into the tables, [2] error
    GramSlot* gram[ANPD_N_MAX + 1];   // indexed by n
    PrefSlot* pref[ANPD_N_MAX + 1];
    int n_min, n_max, max_ctx, cap, policy;
};

struct anpd_ngram {
    NgramDev h;            // host copy of the descriptor (device pointers inside)
    NgramDev* d;           // device copy, for kernels that take an array of descriptors
    cudaStream_t stream;
    int n_tokens;          // host mirror, valid whenever no asynchronous loop is running
    int n_folded;          // host mirror of state[1]: tokens below it are in the tables
    int* pinned;           // small pinned staging buffer
    void* slab;            // all tables, one allocation
    size_t slab_bytes;
};

// on: the stream to launch on (null: the context's own)
anpd_status ngram_enqueue_bulk(anpd_ngram* ctx, int from, int to, Profiler* prof, cudaStream_t on = nullptr);
// One fused launch for `batch` sequences: folds tokens [state[1], state[0]) of each, then drafts
// K tokens into seq[b] (draft, draft_len, last_tok).
// K2 > 0: also draft a second candidate of up to K2 tokens into seq[b].draft2
anpd_status ngram_enqueue_step(const NgramDev* d_ctxs, SeqState* d_seq, int batch, int K,
                               cudaStream_t st, Profiler* prof, int K2 = 0);

// proj_rr.cu: the projections of a single-sequence step with their epilogues fused in ("row-range" kernel: each
// CTA owns a contiguous range of output features and the whole contraction dimension).
struct RRPlan {
    int N, K;
    int pairs;             // feature pairs, cut evenly across the CTAs
    int G;                 // CTAs
    int r_max;             // most features a CTA owns (even)
    int mt;                // features per epilogue thread (1 or 2)
    int P;                 // 16-wide slices of K packed into one MMA (1, 2, 4 or 8; P * r_max <= 256)
    int k_blocks, kb, n_stages, stages;
    int w_step_stride, w_step_global, a_off, stage_bytes, scratch_off, smem_bytes;
    int rotate, one_copy;
    unsigned long long slot_bytes;
};
struct RRPlanDev { int G, pairs, r_max, kb, n_stages, rotate, P, w_step_global; unsigned long long slot_bytes; };
// Stage at which CTA c of G starts its walk over the n_stages stages of K (it wraps around).
__host__ __device__ inline int rr_rotation(int c, int G, int n_stages) { return (int)((long long)c * n_stages / G); }
enum RREpilogue { RR_RAW = 0, RR_QKV = 1, RR_RESID = 2, RR_GU = 3, RR_LM = 4 };
enum RRRowMap { RR_MAP_IDENTITY = 0, RR_MAP_HEADS = 1, RR_MAP_GATE_UP = 2 };
// Operand image of the activations of a single-sequence step: per 64-wide k-block 64 operand rows of 32 bytes
// (row = 16 * slice + term, slice = the 16-wide part of the k-block, terms 0-7 = hi parts of the step's rows, 8-15 = lo
// parts) in the 32-byte-swizzled K-major layout.  Byte offset of element (term row16, k):
__host__ __device__ inline size_t act_img_offset(int row16, int k) {
    const int R = ((k >> 4) & 3) * 16 + row16;
    return (size_t)(k >> 6) * 2048 + (size_t)R * 32 + (size_t)(((((k >> 3) & 1) ^ ((R >> 2) & 1))) << 4) + (size_t)(k & 7) * 2;
}
// one k-block more than K needs, left zero: an instruction that packs eight slices spans two k-blocks
inline size_t act_img_bytes(int K) { return (size_t)((K + 63) / 64 + 1) * 2048; }
struct RREpiHost {         // epilogue arguments; only the fields of the chosen epilogue are read
    const float* ss_in = nullptr; int n_parts_in = 0; float inv_d_in = 0; float eps = 0;
    const int* row_pos = nullptr; const int* row_seq = nullptr; const int* row_ok = nullptr;
    const float* rope_cos = nullptr; const float* rope_sin = nullptr; const int* page_table = nullptr;
    int pages_per_seq = 0, Hq = 0, Hkv = 0, hd = 0; float q_scale = 0;
    __nv_bfloat16 *q_hi = nullptr, *q_lo = nullptr, *kpool_l = nullptr, *vpool_l = nullptr;
    float* x = nullptr; const float* gain = nullptr; float* ss_out = nullptr; int d = 0;
    unsigned char* act_out = nullptr;
    float* logits = nullptr; float* amax_val = nullptr; int* amax_idx = nullptr; int V = 0;
    float* raw_out = nullptr;
};
void rr_make_plan(RRPlan* p, int N, int K, int num_sms);
size_t rr_storage_bytes(const RRPlan& p);
anpd_status rr_retile_enqueue(const RRPlan& p, const void* src, bool src_is_f32, int rows, int row_off, int map, int hd, int F,
                              unsigned char* dst, cudaStream_t st);
anpd_status rr_act_image_enqueue(const float* a_dev, int K, unsigned char* img, cudaStream_t st);
anpd_status rr_enqueue(int epi, const RRPlan& p, const unsigned char* w, const unsigned char* act, const RREpiHost& h, int* err,
                       cudaStream_t st, Profiler* prof);

// ---------------------------------------------------------------------------------------------
// model, KV cache and workspace
// ---------------------------------------------------------------------------------------------
constexpr int KV_PAGE = 128;          // positions per KV page (= key chunk of one attention block)
constexpr int PREFILL_ROWS_MAX = 2048; // most rows of one prompt pass (sizes the workspace); a longer prompt takes several passes

// How one [N][K] weight matrix is cut across the persistent GEMM CTAs (depends on the shape and the
// SM count only): tile t is started by CTA first_cta[t] and covered by seg_count[t] consecutive CTAs,
// each of which leaves one partial sum; consumers add them in that order.
struct GemmPlan {
    int N, K, m_tiles, k_blocks, grid, max_segs;
    int max_count;                    // most (tile, k-block) blocks any CTA owns
    std::vector<int> first_cta, seg_count;
    int* d_first_cta;
    int* d_seg_count;
};
enum GemmKind { GK_QKV = 0, GK_O = 1, GK_GU = 2, GK_DOWN = 3, GK_LM = 4, GK_COUNT = 5 };

struct LayerW {
    // all four matrices in tiled storage (see gemm_tiled_elems)
    const __nv_bfloat16* wqkv;        // [(Hq + 2 Hkv) * hd, d]  (q rows, then k rows, then v rows)
    const __nv_bfloat16* wo;          // [d, Hq * hd]
    const __nv_bfloat16* wgu;         // [2 F, d]  (gate rows, then up rows)
    const __nv_bfloat16* wd;          // [d, F]
    const float* attn_norm;           // [d]
    const float* ffn_norm;            // [d]
};

struct anpd_model {
    anpd_model_config cfg;
    cudaStream_t stream;
    int dq, dkv, nqkv;
    const __nv_bfloat16* embed;       // [V, d]
    const __nv_bfloat16* lm_head;     // [V, d], tiled storage
    const float* final_norm;          // [d]
    std::vector<LayerW> layers;
    void* slab;
    size_t slab_bytes;
    double streamed_bytes;            // weight bytes one forward reads
    GemmPlan plan[GK_COUNT];
    int* d_plan_tables;               // device copies of the plans' tables
    int* d_ones;                      // [tiles] all 1: segment counts of the plain GEMM
    int* d_const_segs[4];             // [tiles] all k (k = 1..3): segment counts of a prompt-pass GEMM cut into k parts along K
    int* d_tail_segs[GK_COUNT];       // [tiles] segment counts of a prompt-pass GEMM whose last tiles alone are cut (PfSchedule)
    int tail_cfg[GK_COUNT];           // what d_tail_segs[kind] holds: first cut feature tile * 4 + parts, -1 = nothing yet
    int max_segs;
    bool plain_gemm;                  // debugging aid: route GEMMs through the plain kernel
    // second copy of the projections in row-range storage, used by single-sequence steps (proj_rr.cu)
    RRPlan rr[GK_COUNT];
    struct LayerRR { const unsigned char *wqkv, *wo, *wgu, *wd; };
    std::vector<LayerRR> rr_layers;
    const unsigned char* rr_lm;
    void* rr_slab;
    bool rr_ready;
    int num_sms;
    int device;                       // ordinal of the device the weight blocks were laid out for
    Profiler prof;
};

struct Workspace {
    int r_max;                        // rows any forward may use
    int prefill_rows;                 // rows of one prompt pass (a multiple of 256)
    int n_max_out;                    // widest GEMM output (max of nqkv, 2F, d, V)
    int splits_max;
    int* row_tok; int* row_pos; int* row_seq; int* row_ok;    // [r_max]
    // two-candidate mode: the cache slot a row's K/V go to (its position otherwise) and a range of slots it must not see
    int* row_slot; int* row_hole_lo; int* row_hole_hi;          // [r_max]
    float* x;                         // [r_max, d] residual stream
    __nv_bfloat16 *h_hi, *h_lo;       // [r_max, d]   normalised input of QKV / gate-up / LM head
    __nv_bfloat16 *ao_hi, *ao_lo;     // [r_max, dq]  attention output, input of the O projection
    __nv_bfloat16 *act_hi, *act_lo;   // [r_max, F]   SwiGLU output, input of the down projection
    float* part;                      // [splits_max, r_max, n_max_out] GEMM partial sums
    __nv_bfloat16 *q_hi, *q_lo;       // [r_max, dq] rotated queries x log2(e)/sqrt(hd), as two bf16 terms
    float *attn_m, *attn_l, *attn_o;  // per (row, q head, key chunk): max, sum, weighted values
    float* logits;                    // [r_max, V]
    float* amax_val; int* amax_idx;   // [r_max, amax_blocks]
    int amax_blocks;
    // single-sequence steps: operand images of the four projection inputs, partial sums of squares of the residual
    // stream ([CTA][8 rows]; a: after the down projection / embedding, b: after the O projection), per-CTA argmax
    unsigned char *img_h, *img_h2, *img_ao, *img_act;
    float *ss_a, *ss_b;
    float* amax_val_rr; int* amax_idx_rr;
    int amax_nblk;                    // argmax candidates per row left by the last forward (depends on the path it took)
    float* amax_val_use; int* amax_idx_use;   // ... and the arrays that hold them
    int* gemm_err;                    // device flag set by a GEMM kernel that gave up waiting
    // TMA views of the activation buffers: [0] decode (batch*8 rows), [1] prompt passes (prefill_rows rows, boxes of 128 rows)
    CUtensorMap map_h[2][2], map_ao[2][2], map_act[2][2];     // [mode][hi/lo]
    CUtensorMap map_q[2];             // the queries of a prompt pass (hi, lo) through boxes of 64 columns x 128 rows (head dimension 128)
    int nb[2];                        // MMA N per mode (rows padded to a multiple of 16)
};

// Arguments of the persistent step kernel (step_kernel.cu), fixed for a (model, cache) pair.
struct StepGemm {
    int N, K, m_tiles, k_blocks, grid;
    const int* first_cta;             // [m_tiles] CTA that owns a tile's first k-block
    const int* seg_count;             // [m_tiles] partial sums that cover the tile
    float* part;                      // [segment][row][ld_part], one buffer per projection kind
    unsigned long long seg_stride;
    int ld_part;
};
struct StepLayer { const __nv_bfloat16 *wqkv, *wo, *wgu, *wd; const float *attn_norm, *ffn_norm; };
struct StepParams {
    alignas(64) CUtensorMap map_k, map_v;
    StepGemm g[5];
    const StepLayer* layers;
    const __nv_bfloat16 *embed, *lm_head;
    const float* final_norm;
    int L, d, F, V, Hq, Hkv, hd, dq, rows, stages;
    float eps, q_scale;
    const int *row_tok, *row_pos, *row_seq, *row_ok;
    float* x;
    // operand images of the projections' inputs (see img_offset in step_kernel.cu): QKV / LM head, gate/up, O, down
    unsigned char *imgA, *imgB, *img_ao, *img_act;
    __nv_bfloat16 *q_hi, *q_lo;
    float *ssA, *ssB;                     // [d / 128][rows] sums of squares of the residual stream per 128-column tile
    float *pm, *pl, *po;                  // attention page partials
    float* logits; float* amax_val; int* amax_idx;
    __nv_bfloat16 *kpool, *vpool;
    unsigned long long layer_elems;       // elements of one layer of a pool
    int layer_rows;                       // rows of one layer in the pools' 2-D view
    const int* page_table; int pages_per_seq;
    const float *rope_cos, *rope_sin;
    // phase and arrival counters, zeroed before every step: (L + 1) blocks of `sync_stride` ints
    int* sync; int sync_stride;
    int o_dh, o_dqkv, o_dao, o_dhB, o_dact, o_ditems;            // phase counters: finished tiles of the phase that writes hA / q,k,v / ao / hB / act
    int o_cqkv, o_cattn, o_co, o_cgu, o_cdown, o_clm;   // per-tile arrival counters
    int* err;
    unsigned long long* trace;            // optional time stamps (debugging aid), or null
    int trace_cta;
};

struct anpd_kv {
    anpd_model* m;
    int batch, max_len, pages_per_seq, total_pages;
    __nv_bfloat16 *kpool, *vpool;     // per layer and page: K [Hkv][KV_PAGE][hd]; V transposed [Hkv][hd][KV_PAGE]
    CUtensorMap map_k, map_v;         // TMA views of the two pools as [all page rows][hd] matrices (head dimension 128 only)
    bool attn_tc;                     // attention on tcgen05 (head dimension 128); otherwise the mma.sync kernel
    bool attn_pf;                     // prompt passes: the 128-row kernel (attn_pf.cu); otherwise the 16-row kernel of attn_tc.cu
    int* page_table;                  // device [batch][pages_per_seq]
    float *rope_cos, *rope_sin;       // [max_len][hd/2]
    SeqState* seq;                    // device [batch]
    SeqState* h_seq;                  // pinned host staging [batch]
    int* d_prompt;                    // device [max_len]
    NgramDev* d_ctxs;                 // device [batch]: descriptors of the sequences' n-gram contexts
    int* h_small;                     // pinned, a few ints
    std::vector<int> h_kv_len;        // host mirror of the sequences' lengths
    std::vector<char> h_len_stale;    // a committing step was enqueued and its outcome not read yet: the mirror is behind
    Workspace ws;
    void* slab;
    size_t slab_bytes;
    bool staged;
    int candidates;                   // 1, or 2: every step of the decoding loop verifies a second candidate too
    // one instantiated CUDA graph per distinct step shape (draft length, mode, attention grid)
    struct StepGraph { cudaGraphExec_t exec; int launches; };
    std::map<uint64_t, StepGraph> graphs;
    // the device-resident decoding loop: one graph (a WHILE node around the step) per (draft length, context bound)
    std::map<uint64_t, StepGraph> loop_graphs;
    bool loop_ok;                     // false once building such a graph has failed, or when ANPD_HOST_LOOP is set
    int* loop_steps_left;             // device: steps the running loop may still take
    // Initialize (the prompt's n-gram statistics) runs on a stream of its own under the prompt passes
    cudaStream_t side_stream;
    cudaEvent_t ev_fork, ev_join;
    int loop_launches_per_step;
    // persistent step kernel: its arguments, the buffers only it uses, and whether decode steps take it
    StepParams step;
    bool step_ready;
    void* step_slab;                  // second gate/up input, per-projection partial sums, tile sums of squares, flags, layer table
    size_t step_sync_bytes;
    int step_smem;
    bool use_graphs;
    bool warm;                       // the first step runs eagerly (one-time function attributes, lazy module loading)
};

// Forward over `rows` rows (a multiple of 8; 8 consecutive rows always belong to one sequence and
// hold consecutive positions).  The row plan (ws.row_*) must have been written on the stream.
// max_pos: an upper bound of the largest position any row holds (sizes the attention grid).
// head: also run the LM head and the per-block argmax (false for all but the last prefill pass).
// head_row: in a prompt pass, the row whose next token is wanted (the LM head runs for its group of 8 rows only).
anpd_status forward_enqueue(anpd_model* m, anpd_kv* kv, int rows, int max_pos, bool head, bool want_logits, int head_row = 0, bool two_candidates = false);

// step_kernel.cu: the whole forward of a decode step as ONE persistent kernel (one CTA per SM).  True if this model / cache
// pair can take that path (head dimension 128, one query head per kv head, dimensions that are multiples of 128).
bool step_kernel_eligible(const anpd_model* m, const anpd_kv* kv);
anpd_status step_kernel_setup(anpd_model* m, anpd_kv* kv);              // fills kv->step (buffers are part of the kv slab)
anpd_status step_kernel_enqueue(anpd_model* m, anpd_kv* kv, int max_pos, bool want_logits);
void step_kernel_trace_dump(anpd_kv* kv);

enum AcceptMode { ACCEPT_COMMIT = 0, ACCEPT_PEEK = 1, ACCEPT_PREFILL = 2 };
anpd_status plan_decode_enqueue(anpd_model* m, anpd_kv* kv, bool two_candidates = false);
anpd_status plan_prefill_enqueue(anpd_model* m, anpd_kv* kv, int seq, int start, int prompt_len, int rows);
// mode COMMIT/PEEK: one block per sequence over its 8 rows.  PREFILL: `last_row` of sequence
// `seq` gives the first generated token, kv_len becomes prompt_len.  d_ctxs may be null; otherwise
// accepted tokens and the next token are appended to the sequences' token buffers.
anpd_status accept_enqueue(anpd_model* m, anpd_kv* kv, int mode, const NgramDev* d_ctxs, int seq, int last_row, int prompt_len, bool two_candidates = false);

// attn_tc.cu: per-page attention partials for head dimension 128 (same outputs as the mma.sync kernel in forward.cu)
// tree: the rows carry cache slots and hidden slot ranges of their own (two-candidate steps)
anpd_status attn_tc_enqueue(anpd_model* m, anpd_kv* kv, int layer, int rows, int max_pos, bool tree = false);
// attn_pf.cu: attention of a prompt pass with 128 query rows per CTA (head dimension 128, one query head per kv head)
anpd_status attn_pf_enqueue(anpd_model* m, anpd_kv* kv, int layer, int rows);
// attention of a prompt pass (one query head per kv head), written straight to the O projection's input
anpd_status attn_prompt_enqueue(anpd_model* m, anpd_kv* kv, int layer, int rows);

// gemm_tc.cu
anpd_status make_tmap_bf16(CUtensorMap* out, const void* base, int rows, int K, int box_rows, bool streamed);
// Weight matrices are stored as 128 x 64 blocks of 16 KB.  The GEMM's CTA c owns the logical blocks
// [c * total / G, (c + 1) * total / G) (logical index = tile * k_blocks + k_block) and reads its i-th
// block at step i; that block is stored in slot i * G + c.  So at every step the G CTAs together read
// one contiguous window of G * 16 KB, and the window sweeps through memory like a plain copy would.
__host__ __device__ inline long long gemm_block_slot(long long logical, long long total, int G) {
    const long long c = ((logical + 1) * G + total - 1) / total - 1;      // owner: largest c with c * total / G <= logical
    return (logical - c * total / G) * G + c;
}
// Inside its 16 KB slot a block is stored as the shared-memory image the MMA reads: rows of 128 bytes, and
// within every group of 8 rows the 16-byte chunk c of row r sits at chunk position c ^ (r % 8) (the 128-byte
// swizzle).  The GEMM brings a block in with one linear copy.  Element (row r, column k) of a block:
__host__ __device__ inline size_t gemm_block_elem(long long slot, int r, int k) {
    return ((size_t)slot * 128 + r) * 64 + (size_t)((((k >> 3) ^ (r & 7)) << 3) | (k & 7));
}
void gemm_make_plan(GemmPlan* p, int N, int K, int num_sms);
size_t gemm_tiled_elems(const GemmPlan& p);
// Scatters rows [row_off, row_off + rows) of a row-major [rows][K] source (bf16, or fp32 rounded to
// bf16) into the block storage of the plan's matrix.  The padding must already be zero.
anpd_status gemm_retile_enqueue(const GemmPlan& p, const void* src, bool src_is_f32, int rows, int row_off, __nv_bfloat16* dst_tiled, cudaStream_t st);
anpd_status gemm_tc_enqueue(const GemmPlan& plan, const __nv_bfloat16* w_blocks, const CUtensorMap& map_hi, const CUtensorMap& map_lo,
                            int rows, int NB, float* part, size_t seg_stride, int ld_part, int* err, cudaStream_t st,
                            Profiler* prof);
// gemm_pf.cu: the projection of a prompt pass (many rows, bound by the tensor cores): out[row][n], complete sums
// out[part][row][n]: partial sums per output, seg_stride elements apart.  How the output tiles (feature pair x row tile, row
// tile fastest) are cut along K: tiles [0, tail_from) into `ksplit` equal parts each, tiles [tail_from, end) - those that would
// form a last, partly filled round of CTAs - into `tail_split` parts (tail_from == tile count: no such tail; a multiple of the
// row tile count, so that a feature tile has one part count for all its rows).
struct PfSchedule { int ksplit, tail_from, tail_split; };
PfSchedule gemm_pf_schedule(int n_ft, int n_tt, int k_blocks, int num_sms);
anpd_status gemm_pf_enqueue(const GemmPlan& plan, const __nv_bfloat16* w_blocks, const CUtensorMap& map_hi, const CUtensorMap& map_lo, int rows,
                            float* out, int ld, size_t seg_stride, PfSchedule sched, int num_sms, int* err, cudaStream_t st, Profiler* prof);
// forward.cu: the plain (one warp per output feature) GEMM, kept as a cross-check
anpd_status gemm_plain_enqueue(const GemmPlan& p, const __nv_bfloat16* W, const __nv_bfloat16* a_hi, const __nv_bfloat16* a_lo, int rows,
                               float* part, int ld_part, cudaStream_t st, Profiler* prof);
