// Verification forward of a LLaMA-style decoder over the rows of one step against the paged KV
// cache (paper Section 3.1, "Verification": one forward over the K+1 tokens), and the fused
// argmax / draft-compare / prefix-accept that ends the step (Algorithm 1's accept loop).
//
// Row-count invariance: every value a row produces depends on that row's inputs and absolute
// position only - never on how many rows share the launch, nor on which of them are real.  A
// greedy step (1 real row) and an ANPD step (K+1 real rows) therefore give bit-identical logits
// for the same position, which is what makes the two token streams identical.
#include "internal.h"

#include <math_constants.h>

typedef __nv_bfloat16 bf16;

namespace {

constexpr int ERR_TOKEN_RANGE = 101;
constexpr int ERR_KV_FULL = 102;
constexpr int ERR_CTX_FULL = 103;

__device__ __forceinline__ void split_bf16(float v, bf16& hi, bf16& lo) {
    hi = __float2bfloat16_rn(v);
    lo = __float2bfloat16_rn(v - __bfloat162float(hi));
}

// Sum over a 256-thread block in a fixed order (xor-shuffle tree per warp, then across warps).
__device__ __forceinline__ float block_sum_256(float v, float* red /*[8]*/) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = (threadIdx.x & 31) < 8 ? red[threadIdx.x & 31] : 0.0f;
    for (int o = 4; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    t = __shfl_sync(0xffffffffu, t, 0);
    __syncthreads();
    return t;
}

// ---------------------------------------------------------------------------------------------
// row plans
// ---------------------------------------------------------------------------------------------
__global__ void plan_decode_kernel(SeqState* seqs, int* row_tok, int* row_pos, int* row_seq, int* row_ok,
                                   int vocab, int max_len) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const int b = i / ANPD_ROWS, r = i % ANPD_ROWS;
    SeqState& s = seqs[b];
    int tok = (r == 0) ? s.last_tok : (r <= s.draft_len ? s.draft[r - 1] : 0);
    if (tok < 0 || tok >= vocab) { if (r <= s.draft_len) atomicExch(&s.error, ERR_TOKEN_RANGE); tok = 0; }
    const int pos = s.kv_len + r;
    if (pos >= max_len && r <= s.draft_len && s.active) atomicExch(&s.error, ERR_KV_FULL);
    row_tok[i] = tok;
    row_pos[i] = min(pos, max_len - 1);
    row_seq[i] = b;
    row_ok[i] = (pos < max_len) ? 1 : 0;
}

__global__ void plan_prefill_kernel(const int* prompt, int seq, int start, int prompt_len, int rows,
                                    int* row_tok, int* row_pos, int* row_seq, int* row_ok, int vocab, int max_len,
                                    SeqState* seqs) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows) return;
    const int p = start + i;
    int tok = (p < prompt_len) ? prompt[p] : 0;
    if (tok < 0 || tok >= vocab) { atomicExch(&seqs[seq].error, ERR_TOKEN_RANGE); tok = 0; }
    row_tok[i] = tok;
    row_pos[i] = min(p, max_len - 1);
    row_seq[i] = seq;
    row_ok[i] = (p < max_len && p < prompt_len) ? 1 : 0;
}

// ---------------------------------------------------------------------------------------------
// embedding gather + first RMSNorm;  residual add + RMSNorm
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) embed_norm_kernel(const bf16* __restrict__ embed, const int* __restrict__ row_tok,
                                                         const float* __restrict__ gain, float eps, int d,
                                                         float* __restrict__ x, bf16* __restrict__ h_hi, bf16* __restrict__ h_lo) {
    __shared__ float red[8];
    const int row = blockIdx.x;
    const bf16* e = embed + (size_t)row_tok[row] * d;
    float* xr = x + (size_t)row * d;
    float ss = 0.0f;
    for (int i = threadIdx.x; i < d; i += 256) {
        const float v = __bfloat162float(e[i]);
        xr[i] = v;
        ss += v * v;
    }
    const float rstd = rsqrtf(block_sum_256(ss, red) / (float)d + eps);
    for (int i = threadIdx.x; i < d; i += 256) {
        bf16 hi, lo;
        split_bf16(xr[i] * rstd * gain[i], hi, lo);
        h_hi[(size_t)row * d + i] = hi;
        h_lo[(size_t)row * d + i] = lo;
    }
}

// x[row] += sum over splits of part[s][row]; then h = rmsnorm(x) * gain, split into hi + lo.
__global__ void __launch_bounds__(256) resid_norm_kernel(float* __restrict__ x, const float* __restrict__ part, const int* __restrict__ seg_count,
                                                         size_t split_stride, int ld_part, const float* __restrict__ gain,
                                                         float eps, int d, bf16* __restrict__ h_hi, bf16* __restrict__ h_lo) {
    __shared__ float red[8];
    const int row = blockIdx.x;
    float* xr = x + (size_t)row * d;
    float ss = 0.0f;
    for (int i = threadIdx.x; i < d; i += 256) {
        float v = xr[i];
        const int ns = seg_count[i >> 7];
        for (int s = 0; s < ns; ++s) v += part[s * split_stride + (size_t)row * ld_part + i];
        xr[i] = v;
        ss += v * v;
    }
    const float rstd = rsqrtf(block_sum_256(ss, red) / (float)d + eps);
    for (int i = threadIdx.x; i < d; i += 256) {
        bf16 hi, lo;
        split_bf16(xr[i] * rstd * gain[i], hi, lo);
        h_hi[(size_t)row * d + i] = hi;
        h_lo[(size_t)row * d + i] = lo;
    }
}

// ---------------------------------------------------------------------------------------------
// QKV epilogue: reduce splits, rotary embedding, append K/V to the paged cache, keep q
// ---------------------------------------------------------------------------------------------
__global__ void qkv_rope_append_kernel(const float* __restrict__ part, const int* __restrict__ seg_count, size_t split_stride, int ld_part,
                                       const int* __restrict__ row_pos, const int* __restrict__ row_seq,
                                       const int* __restrict__ row_ok, const float* __restrict__ rope_cos,
                                       const float* __restrict__ rope_sin, const int* __restrict__ page_table,
                                       int pages_per_seq, int Hq, int Hkv, int hd, float* __restrict__ q,
                                       bf16* __restrict__ kpool_l, bf16* __restrict__ vpool_l) {
    const int row = blockIdx.x, head = blockIdx.y, i = threadIdx.x, half = hd >> 1;
    const float* pr = part + (size_t)row * ld_part + (size_t)head * hd;
    float a = 0.0f, b = 0.0f;
    const int ns = seg_count[(head * hd + i) >> 7];      // a head never straddles a 128-column tile
    for (int s = 0; s < ns; ++s) { a += pr[s * split_stride + i]; b += pr[s * split_stride + i + half]; }
    const int pos = row_pos[row];
    if (head < Hq + Hkv) {
        const float c = rope_cos[(size_t)pos * half + i], sn = rope_sin[(size_t)pos * half + i];
        const float ra = a * c - b * sn, rb = b * c + a * sn;
        a = ra; b = rb;
    }
    if (head < Hq) {
        q[(size_t)row * Hq * hd + head * hd + i] = a;
        q[(size_t)row * Hq * hd + head * hd + i + half] = b;
        return;
    }
    if (!row_ok[row]) return;
    const bool is_k = head < Hq + Hkv;
    const int kvh = is_k ? head - Hq : head - Hq - Hkv;
    const int page = page_table[row_seq[row] * pages_per_seq + pos / KV_PAGE];
    bf16* dst = (is_k ? kpool_l : vpool_l) + (((size_t)page * Hkv + kvh) * KV_PAGE + (pos % KV_PAGE)) * hd;
    dst[i] = __float2bfloat16_rn(a);
    dst[i + half] = __float2bfloat16_rn(b);
}

// ---------------------------------------------------------------------------------------------
// attention: per (key page, kv head, group of 8 rows) partial softmax, then a combine in page order
// ---------------------------------------------------------------------------------------------
template <int HD>
__global__ void __launch_bounds__(256) attn_partial_kernel(const float* __restrict__ q, const bf16* __restrict__ kpool_l,
                                                           const bf16* __restrict__ vpool_l, const int* __restrict__ page_table,
                                                           int pages_per_seq, const int* __restrict__ row_pos,
                                                           const int* __restrict__ row_seq, int Hq, int Hkv, float scale,
                                                           float* __restrict__ pm, float* __restrict__ pl, float* __restrict__ po) {
    constexpr int KP = HD + 8;                 // padded K row (elements): 16-byte reads stay conflict-free
    extern __shared__ __align__(16) unsigned char smem[];
    const int G = Hq / Hkv, NQ = ANPD_ROWS * G;
    bf16* Ks = (bf16*)smem;                                   // [KV_PAGE][KP]
    bf16* Vs = Ks + KV_PAGE * KP;                             // [KV_PAGE][HD]
    float* qs = (float*)(Vs + KV_PAGE * HD);                  // [NQ][HD]
    float* S = qs + NQ * HD;                                  // [NQ][KV_PAGE]

    const int c = blockIdx.x, g = blockIdx.y, r0 = blockIdx.z * ANPD_ROWS;
    const int pos_lo = row_pos[r0], pos_hi = row_pos[r0 + ANPD_ROWS - 1];
    if (c * KV_PAGE > pos_hi) return;
    const int n_keys = min(KV_PAGE, pos_hi - c * KV_PAGE + 1);
    const int page = page_table[row_seq[r0] * pages_per_seq + c];
    const bf16* Kg = kpool_l + ((size_t)page * Hkv + g) * KV_PAGE * HD;
    const bf16* Vg = vpool_l + ((size_t)page * Hkv + g) * KV_PAGE * HD;
    const int tid = threadIdx.x;

    constexpr int VPR = HD / 8;                // 16-byte vectors per row
    for (int v = tid; v < n_keys * VPR; v += 256) {
        const int j = v / VPR, w = v % VPR;
        *(uint4*)(Ks + j * KP + w * 8) = *(const uint4*)(Kg + (size_t)j * HD + w * 8);
        *(uint4*)(Vs + j * HD + w * 8) = *(const uint4*)(Vg + (size_t)j * HD + w * 8);
    }
    for (int v = tid; v < NQ * HD; v += 256) {
        const int qi = v / HD, dim = v % HD;
        const int r = qi / G, hl = qi % G;
        qs[v] = q[(size_t)(r0 + r) * Hq * HD + (g * G + hl) * HD + dim] * scale;
    }
    __syncthreads();

    // scores: thread = (key j, half of the query vectors), four query vectors at a time
    {
        const int j = tid & (KV_PAGE - 1), part = tid >> 7;
        const int q_lo = part * (NQ / 2), q_hi = q_lo + NQ / 2;
        const int key_pos = c * KV_PAGE + j;
        for (int qb = q_lo; qb < q_hi; qb += 4) {
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            if (j < n_keys) {
                for (int w = 0; w < VPR; ++w) {
                    const uint4 kv = *(const uint4*)(Ks + j * KP + w * 8);
                    const bf16* k8 = (const bf16*)&kv;
                    float kf[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) kf[e] = __bfloat162float(k8[e]);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const float4 qa = *(const float4*)(qs + (qb + u) * HD + w * 8);
                        const float4 qc = *(const float4*)(qs + (qb + u) * HD + w * 8 + 4);
                        float a = acc[u];
                        a = fmaf(qa.x, kf[0], a); a = fmaf(qa.y, kf[1], a); a = fmaf(qa.z, kf[2], a); a = fmaf(qa.w, kf[3], a);
                        a = fmaf(qc.x, kf[4], a); a = fmaf(qc.y, kf[5], a); a = fmaf(qc.z, kf[6], a); a = fmaf(qc.w, kf[7], a);
                        acc[u] = a;
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int r = (qb + u) / G;
                const bool visible = (j < n_keys) && (key_pos <= pos_lo + r);
                S[(qb + u) * KV_PAGE + j] = visible ? acc[u] : -CUDART_INF_F;
            }
        }
    }
    __syncthreads();

    // softmax pieces per query vector: one warp each, fixed reduction tree
    {
        const int warp = tid >> 5, lane = tid & 31;
        for (int qi = warp; qi < NQ; qi += 8) {
            float* s = S + qi * KV_PAGE;
            float m = -CUDART_INF_F;
            for (int j = lane; j < KV_PAGE; j += 32) m = fmaxf(m, s[j]);
            for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            float l = 0.0f;
            for (int j = lane; j < KV_PAGE; j += 32) {
                const float p = (m == -CUDART_INF_F) ? 0.0f : expf(s[j] - m);
                s[j] = p;
                l += p;
            }
            for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
            if (lane == 0) {
                const int r = qi / G, hl = qi % G;
                const size_t idx = ((size_t)(r0 + r) * Hq + (g * G + hl)) * pages_per_seq + c;
                pm[idx] = m;
                pl[idx] = l;
            }
        }
    }
    __syncthreads();

    // weighted values: thread = (pair of dims, subset of query vectors), keys in position order
    {
        constexpr int TPQ = HD / 2;            // threads covering one query vector
        constexpr int QSUB = 256 / TPQ;        // query-vector subsets
        const int dp = tid % TPQ, sub = tid / TPQ;
        for (int qi = sub; qi < NQ; qi += QSUB) {
            float o0 = 0.0f, o1 = 0.0f;
            const float* s = S + qi * KV_PAGE;
            for (int j = 0; j < n_keys; ++j) {
                const __nv_bfloat162 v2 = *(const __nv_bfloat162*)(Vs + j * HD + 2 * dp);
                const float p = s[j];
                o0 = fmaf(p, __low2float(v2), o0);
                o1 = fmaf(p, __high2float(v2), o1);
            }
            const int r = qi / G, hl = qi % G;
            const size_t idx = ((size_t)(r0 + r) * Hq + (g * G + hl)) * pages_per_seq + c;
            po[idx * HD + 2 * dp] = o0;
            po[idx * HD + 2 * dp + 1] = o1;
        }
    }
}

// One block per (row, q head): fold the pages 0..pos/KV_PAGE in order, write the output as hi+lo.
__global__ void attn_combine_kernel(const float* __restrict__ pm, const float* __restrict__ pl, const float* __restrict__ po,
                                    const int* __restrict__ row_pos, int Hq, int hd, int pages_per_seq,
                                    bf16* __restrict__ ao_hi, bf16* __restrict__ ao_lo) {
    const int row = blockIdx.x, head = blockIdx.y, dim = threadIdx.x;
    const int nc = row_pos[row] / KV_PAGE + 1;
    const size_t base = ((size_t)row * Hq + head) * pages_per_seq;
    float M = -CUDART_INF_F;
    for (int c = 0; c < nc; ++c) M = fmaxf(M, pm[base + c]);
    float L = 0.0f, o = 0.0f;
    for (int c = 0; c < nc; ++c) {
        const float w = expf(pm[base + c] - M);
        L = fmaf(pl[base + c], w, L);
        o = fmaf(po[(base + c) * hd + dim], w, o);
    }
    bf16 hi, lo;
    split_bf16(o / L, hi, lo);
    const size_t out = (size_t)row * Hq * hd + head * hd + dim;
    ao_hi[out] = hi;
    ao_lo[out] = lo;
}

// ---------------------------------------------------------------------------------------------
// SwiGLU epilogue of the gate/up projection
// ---------------------------------------------------------------------------------------------
__global__ void swiglu_kernel(const float* __restrict__ part, const int* __restrict__ seg_count, size_t split_stride, int ld_part, int F,
                              bf16* __restrict__ act_hi, bf16* __restrict__ act_lo) {
    const int row = blockIdx.y, j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= F) return;
    const float* pr = part + (size_t)row * ld_part;
    float gte = 0.0f, up = 0.0f;
    const int ng = seg_count[j >> 7], nu = seg_count[(F + j) >> 7];
    for (int s = 0; s < ng; ++s) gte += pr[s * split_stride + j];
    for (int s = 0; s < nu; ++s) up += pr[s * split_stride + F + j];
    const float v = gte / (1.0f + expf(-gte)) * up;
    bf16 hi, lo;
    split_bf16(v, hi, lo);
    act_hi[(size_t)row * F + j] = hi;
    act_lo[(size_t)row * F + j] = lo;
}

// ---------------------------------------------------------------------------------------------
// LM-head epilogue: reduce splits, (optionally) keep logits, per-block argmax with ties to the lowest id
// ---------------------------------------------------------------------------------------------
constexpr int AMAX_COLS = 1024;
__global__ void __launch_bounds__(256) argmax_partial_kernel(const float* __restrict__ part, const int* __restrict__ seg_count, size_t split_stride,
                                                             int ld_part, int V, float* __restrict__ logits,
                                                             float* __restrict__ amax_val, int* __restrict__ amax_idx, int nblk) {
    __shared__ float sv[8];
    __shared__ int si[8];
    const int row = blockIdx.y;
    const float* pr = part + (size_t)row * ld_part;
    float best = -CUDART_INF_F;
    int bidx = 0x7fffffff;
    for (int u = 0; u < AMAX_COLS / 256; ++u) {
        const int v = blockIdx.x * AMAX_COLS + u * 256 + threadIdx.x;
        if (v < V) {
            float z = 0.0f;
            const int ns = seg_count[v >> 7];
            for (int s = 0; s < ns; ++s) z += pr[s * split_stride + v];
            if (logits) logits[(size_t)row * V + v] = z;
            if (z > best) { best = z; bidx = v; }       // ascending v: strict > keeps the lowest id
        }
    }
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bidx, o);
        if (ov > best || (ov == best && oi < bidx)) { best = ov; bidx = oi; }
    }
    if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = best; si[threadIdx.x >> 5] = bidx; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w)
            if (sv[w] > best || (sv[w] == best && si[w] < bidx)) { best = sv[w]; bidx = si[w]; }
        amax_val[(size_t)row * nblk + blockIdx.x] = best;
        amax_idx[(size_t)row * nblk + blockIdx.x] = bidx;
    }
}

// Final argmax per row, draft compare, prefix accept, KV commit, token-buffer append.
__global__ void __launch_bounds__(256) accept_kernel(SeqState* seqs, const float* __restrict__ amax_val,
                                                     const int* __restrict__ amax_idx, int nblk, int mode,
                                                     const NgramDev* ctxs, int seq_arg, int last_row, int prompt_len) {
    __shared__ int pred[ANPD_ROWS];
    const int b = (mode == ACCEPT_PREFILL) ? seq_arg : blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    {
        const int row = (mode == ACCEPT_PREFILL) ? (last_row / ANPD_ROWS) * ANPD_ROWS + warp : b * ANPD_ROWS + warp;
        float best = -CUDART_INF_F;
        int bidx = 0x7fffffff;
        for (int i = lane; i < nblk; i += 32) {
            const float v = amax_val[(size_t)row * nblk + i];
            const int id = amax_idx[(size_t)row * nblk + i];
            if (v > best || (v == best && id < bidx)) { best = v; bidx = id; }
        }
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, best, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bidx, o);
            if (ov > best || (ov == best && oi < bidx)) { best = ov; bidx = oi; }
        }
        if (lane == 0) pred[warp] = bidx;
    }
    __syncthreads();
    if (threadIdx.x != 0) return;
    SeqState& s = seqs[b];
    if (mode == ACCEPT_PREFILL) {
        const int nxt = pred[last_row % ANPD_ROWS];
        s.next_tok = nxt;
        s.kv_len = prompt_len;
        s.accepted_len = 0;
        if (ctxs) {
            const NgramDev& c = ctxs[b];
            const int T = c.state[0];
            if (T + 1 > c.max_ctx) { s.error = ERR_CTX_FULL; s.active = 0; return; }
            c.tokens[T] = nxt;
            c.state[0] = T + 1;
        }
        return;
    }
    int a = 0;
    while (a < s.draft_len && s.draft[a] == pred[a]) ++a;
    for (int r = 0; r < ANPD_ROWS; ++r) s.pred[r] = pred[r];
    s.accepted_len = a;
    s.next_tok = pred[a];
    if (mode != ACCEPT_COMMIT || !s.active) return;
    s.kv_len += a + 1;
    s.steps += 1;
    s.drafted += s.draft_len;
    s.accepted += a;
    s.hist[a] += 1;
    if (ctxs) {
        const NgramDev& c = ctxs[b];
        const int T = c.state[0];
        if (T + a + 1 > c.max_ctx) { s.error = ERR_CTX_FULL; s.active = 0; return; }
        for (int i = 0; i < a; ++i) c.tokens[T + i] = s.draft[i];
        c.tokens[T + a] = pred[a];
        c.state[0] = T + a + 1;
        if (T + a + 1 >= s.stop_at) s.active = 0;
    }
}

// ---------------------------------------------------------------------------------------------
// weight-streaming GEMM, plain version: one warp per output feature, 8 rows at a time
//   part[0][row][n] = sum_k W[n][k] * (a_hi[row][k] + a_lo[row][k])
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) gemm_rows8_kernel(const bf16* __restrict__ W, const bf16* __restrict__ a_hi,
                                                         const bf16* __restrict__ a_lo, int rows, int N, int K,
                                                         float* __restrict__ part, int ld_part) {
    const int n = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (n >= N) return;
    const bf16* w = W + (size_t)n * K;
    for (int r0 = 0; r0 < rows; r0 += 8) {
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int k0 = lane * 8; k0 < K; k0 += 256) {
            const uint4 wv = *(const uint4*)(w + k0);
            const bf16* w8 = (const bf16*)&wv;
            float wf[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) wf[e] = __bfloat162float(w8[e]);
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                const uint4 hv = *(const uint4*)(a_hi + (size_t)(r0 + r) * K + k0);
                const uint4 lv = *(const uint4*)(a_lo + (size_t)(r0 + r) * K + k0);
                const bf16* h8 = (const bf16*)&hv;
                const bf16* l8 = (const bf16*)&lv;
                float a = acc[r];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    a = fmaf(wf[e], __bfloat162float(h8[e]), a);
                    a = fmaf(wf[e], __bfloat162float(l8[e]), a);
                }
                acc[r] = a;
            }
        }
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            float a = acc[r];
            for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
            if (lane == 0) part[(size_t)(r0 + r) * ld_part + n] = a;
        }
    }
}

// One projection of the forward.  Returns the per-tile segment counts its consumer must use.
anpd_status gemm_enqueue(anpd_model* m, anpd_kv* kv, int kind, int layer, int rows, const int** seg_count_out) {
    Workspace& ws = kv->ws;
    const GemmPlan& plan = m->plan[kind];
    const int mode = (rows == kv->batch * ANPD_ROWS) ? 0 : 1;
    const bf16* W = kind == GK_LM ? m->lm_head : (kind == GK_QKV ? m->layers[layer].wqkv : kind == GK_O ? m->layers[layer].wo
                                                 : kind == GK_GU ? m->layers[layer].wgu : m->layers[layer].wd);
    const bf16 *a_hi = ws.h_hi, *a_lo = ws.h_lo;
    const CUtensorMap* maps = ws.map_h[mode];
    if (kind == GK_O) { a_hi = ws.ao_hi; a_lo = ws.ao_lo; maps = ws.map_ao[mode]; }
    if (kind == GK_DOWN) { a_hi = ws.act_hi; a_lo = ws.act_lo; maps = ws.map_act[mode]; }
    if (m->plain_gemm) {
        *seg_count_out = m->d_ones;
        return gemm_plain_enqueue(W, a_hi, a_lo, rows, plan.N, plan.K, ws.part, ws.n_max_out, m->stream, &m->prof);
    }
    const CUtensorMap& mw = kind == GK_LM ? m->map_lm : m->layers[layer].map[kind];
    ANPD_TRY(gemm_tc_enqueue(plan, mw, maps[0], maps[1], rows, ws.nb[mode], ws.part, (size_t)ws.r_max * ws.n_max_out,
                             ws.n_max_out, ws.gemm_err, m->stream, &m->prof));
    *seg_count_out = plan.d_seg_count;
    return ANPD_OK;
}

template <int HD>
anpd_status attn_enqueue(anpd_model* m, anpd_kv* kv, int layer, int rows, int max_pos) {
    const anpd_model_config& c = m->cfg;
    Workspace& ws = kv->ws;
    const int G = c.n_q_heads / c.n_kv_heads, NQ = ANPD_ROWS * G;
    const size_t smem = (size_t)KV_PAGE * (HD + 8) * 2 + (size_t)KV_PAGE * HD * 2 + (size_t)NQ * HD * 4 + (size_t)NQ * KV_PAGE * 4;
    static bool attr_set = false;
    if (!attr_set) {
        CUDA_TRY(cudaFuncSetAttribute(attn_partial_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024));
        attr_set = true;
    }
    const size_t layer_elems = (size_t)kv->total_pages * c.n_kv_heads * KV_PAGE * HD;
    const int chunks = max_pos / KV_PAGE + 1;
    dim3 grid(chunks, c.n_kv_heads, rows / ANPD_ROWS);
    LAUNCH(&m->prof, m->stream, KC_ATTN, 0,
           (attn_partial_kernel<HD><<<grid, 256, smem, m->stream>>>(ws.q, kv->kpool + layer * layer_elems, kv->vpool + layer * layer_elems,
                                                                   kv->page_table, kv->pages_per_seq, ws.row_pos, ws.row_seq,
                                                                   c.n_q_heads, c.n_kv_heads, 1.0f / sqrtf((float)HD),
                                                                   ws.attn_m, ws.attn_l, ws.attn_o)));
    LAUNCH(&m->prof, m->stream, KC_ATTN, 0,
           (attn_combine_kernel<<<dim3(rows, c.n_q_heads), HD, 0, m->stream>>>(ws.attn_m, ws.attn_l, ws.attn_o, ws.row_pos, c.n_q_heads,
                                                                              HD, kv->pages_per_seq, ws.ao_hi, ws.ao_lo)));
    return ANPD_OK;
}

}  // namespace

anpd_status gemm_plain_enqueue(const bf16* W, const bf16* a_hi, const bf16* a_lo, int rows, int N, int K, float* part, int ld_part,
                               cudaStream_t st, Profiler* prof) {
    LAUNCH(prof, st, KC_GEMM, 2.0 * (double)N * (double)K,
           (gemm_rows8_kernel<<<(N + 7) / 8, 256, 0, st>>>(W, a_hi, a_lo, rows, N, K, part, ld_part)));
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}

anpd_status plan_decode_enqueue(anpd_model* m, anpd_kv* kv) {
    Workspace& ws = kv->ws;
    LAUNCH(&m->prof, m->stream, KC_OTHER, 0,
           (plan_decode_kernel<<<kv->batch, ANPD_ROWS, 0, m->stream>>>(kv->seq, ws.row_tok, ws.row_pos, ws.row_seq, ws.row_ok,
                                                                      m->cfg.vocab, kv->max_len)));
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}

anpd_status plan_prefill_enqueue(anpd_model* m, anpd_kv* kv, int seq, int start, int prompt_len, int rows) {
    Workspace& ws = kv->ws;
    LAUNCH(&m->prof, m->stream, KC_OTHER, 0,
           (plan_prefill_kernel<<<(rows + 127) / 128, 128, 0, m->stream>>>(kv->d_prompt, seq, start, prompt_len, rows, ws.row_tok,
                                                                          ws.row_pos, ws.row_seq, ws.row_ok, m->cfg.vocab,
                                                                          kv->max_len, kv->seq)));
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}

anpd_status accept_enqueue(anpd_model* m, anpd_kv* kv, int mode, const NgramDev* d_ctxs, int seq, int last_row, int prompt_len) {
    Workspace& ws = kv->ws;
    const int blocks = (mode == ACCEPT_PREFILL) ? 1 : kv->batch;
    LAUNCH(&m->prof, m->stream, KC_OTHER, 0,
           (accept_kernel<<<blocks, 256, 0, m->stream>>>(kv->seq, ws.amax_val, ws.amax_idx, ws.amax_blocks, mode, d_ctxs, seq,
                                                        last_row, prompt_len)));
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}

anpd_status forward_enqueue(anpd_model* m, anpd_kv* kv, int rows, int max_pos, bool head, bool want_logits) {
    const anpd_model_config& c = m->cfg;
    Workspace& ws = kv->ws;
    cudaStream_t st = m->stream;
    Profiler* pf = &m->prof;
    const int d = c.d_model, F = c.d_ffn, hd = c.head_dim, V = c.vocab;
    const size_t sstride = (size_t)ws.r_max * ws.n_max_out;
    const size_t layer_elems = (size_t)kv->total_pages * c.n_kv_heads * KV_PAGE * hd;
    const int* segs = nullptr;

    LAUNCH(pf, st, KC_OTHER, 0, (embed_norm_kernel<<<rows, 256, 0, st>>>(m->embed, ws.row_tok, m->layers[0].attn_norm, c.rms_eps, d,
                                                                      ws.x, ws.h_hi, ws.h_lo)));
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerW& w = m->layers[l];
        ANPD_TRY(gemm_enqueue(m, kv, GK_QKV, l, rows, &segs));
        LAUNCH(pf, st, KC_OTHER, 0,
               (qkv_rope_append_kernel<<<dim3(rows, c.n_q_heads + 2 * c.n_kv_heads), hd / 2, 0, st>>>(
                   ws.part, segs, sstride, ws.n_max_out, ws.row_pos, ws.row_seq, ws.row_ok, kv->rope_cos, kv->rope_sin,
                   kv->page_table, kv->pages_per_seq, c.n_q_heads, c.n_kv_heads, hd, ws.q, kv->kpool + l * layer_elems,
                   kv->vpool + l * layer_elems)));
        if (hd == 128) ANPD_TRY(attn_enqueue<128>(m, kv, l, rows, max_pos));
        else ANPD_TRY(attn_enqueue<64>(m, kv, l, rows, max_pos));
        ANPD_TRY(gemm_enqueue(m, kv, GK_O, l, rows, &segs));
        LAUNCH(pf, st, KC_OTHER, 0,
               (resid_norm_kernel<<<rows, 256, 0, st>>>(ws.x, ws.part, segs, sstride, ws.n_max_out, w.ffn_norm, c.rms_eps, d,
                                                       ws.h_hi, ws.h_lo)));
        ANPD_TRY(gemm_enqueue(m, kv, GK_GU, l, rows, &segs));
        LAUNCH(pf, st, KC_OTHER, 0,
               (swiglu_kernel<<<dim3((F + 255) / 256, rows), 256, 0, st>>>(ws.part, segs, sstride, ws.n_max_out, F, ws.act_hi,
                                                                          ws.act_lo)));
        ANPD_TRY(gemm_enqueue(m, kv, GK_DOWN, l, rows, &segs));
        const float* next_gain = (l + 1 < c.n_layers) ? m->layers[l + 1].attn_norm : m->final_norm;
        LAUNCH(pf, st, KC_OTHER, 0,
               (resid_norm_kernel<<<rows, 256, 0, st>>>(ws.x, ws.part, segs, sstride, ws.n_max_out, next_gain, c.rms_eps, d,
                                                       ws.h_hi, ws.h_lo)));
    }
    if (!head) { CUDA_TRY(cudaGetLastError()); return ANPD_OK; }
    ANPD_TRY(gemm_enqueue(m, kv, GK_LM, 0, rows, &segs));
    LAUNCH(pf, st, KC_OTHER, 0,
           (argmax_partial_kernel<<<dim3(ws.amax_blocks, rows), 256, 0, st>>>(ws.part, segs, sstride, ws.n_max_out, V,
                                                                             want_logits ? ws.logits : nullptr, ws.amax_val,
                                                                             ws.amax_idx, ws.amax_blocks)));
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}
