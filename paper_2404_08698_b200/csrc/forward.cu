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

// ---------------------------------------------------------------------------------------------
// row plans
// ---------------------------------------------------------------------------------------------
// Rows of a sequence's step: row 0 the confirmed token at position P; rows 1..ka the first candidate at positions P+1..;
// with a second candidate (two-candidate mode) rows ka+1..ka+kb hold its tokens at positions P+1.. again, but their K/V go
// to the cache slots behind the first candidate's (slot = P + row), and they must not see the first candidate's slots.
__global__ void plan_decode_kernel(SeqState* seqs, int* row_tok, int* row_pos, int* row_seq, int* row_ok, int* row_slot,
                                   int* row_hole_lo, int* row_hole_hi, int vocab, int max_len, int two) {
    pdl_trigger();
    pdl_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const int b = i / ANPD_ROWS, r = i % ANPD_ROWS;
    SeqState& s = seqs[b];
    const int ka = s.draft_len, kb = two ? min(s.draft2_len, ANPD_K_MAX - ka) : 0;
    const bool real = r <= ka + kb;
    int tok = (r == 0) ? s.last_tok : (r <= ka ? s.draft[r - 1] : (real ? s.draft2[r - ka - 1] : 0));
    if (tok < 0 || tok >= vocab) { if (real) atomicExch(&s.error, ERR_TOKEN_RANGE); tok = 0; }
    const int slot = s.kv_len + r;
    const int pos = (r > ka && real) ? s.kv_len + (r - ka) : slot;
    if (slot >= max_len && real && s.active) atomicExch(&s.error, ERR_KV_FULL);
    row_tok[i] = tok;
    row_pos[i] = min(pos, max_len - 1);
    row_seq[i] = b;
    row_ok[i] = (slot < max_len) ? 1 : 0;
    row_slot[i] = min(slot, max_len - 1);
    row_hole_lo[i] = (r > ka && real) ? s.kv_len + 1 : 0;
    row_hole_hi[i] = (r > ka && real) ? s.kv_len + ka + 1 : 0;
}

__global__ void plan_prefill_kernel(const int* prompt, int seq, int start, int prompt_len, int rows,
                                    int* row_tok, int* row_pos, int* row_seq, int* row_ok, int* row_slot, int* row_hole_lo,
                                    int* row_hole_hi, int vocab, int max_len, SeqState* seqs) {
    pdl_trigger();
    pdl_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows) return;
    const int p = start + i;
    int tok = (p < prompt_len) ? prompt[p] : 0;
    if (tok < 0 || tok >= vocab) { atomicExch(&seqs[seq].error, ERR_TOKEN_RANGE); tok = 0; }
    row_tok[i] = tok;
    row_pos[i] = min(p, max_len - 1);
    row_seq[i] = seq;
    row_ok[i] = (p < max_len && p < prompt_len) ? 1 : 0;
    row_slot[i] = min(p, max_len - 1);
    row_hole_lo[i] = 0;
    row_hole_hi[i] = 0;
}

// ---------------------------------------------------------------------------------------------
// embedding gather + first RMSNorm;  residual add + RMSNorm
// One 1024-thread block per row; every thread owns float4 chunks of the row and issues all of a
// chunk's loads (residual + every partial sum) before using any of them, so the kernel costs about
// one memory round trip.  The sum of squares is reduced in a fixed tree.
// ---------------------------------------------------------------------------------------------
constexpr int NORM_THREADS = 1024;
constexpr int NORM_MAX_CHUNKS = 4;        // float4 chunks per thread: rows up to 16384 wide

__device__ __forceinline__ float block_sum_1024(float v, float* red /*[32]*/) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = red[threadIdx.x & 31];
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    __syncthreads();
    return t;
}

__device__ __forceinline__ void store_split4(const float4 v, bf16* hi_ptr, bf16* lo_ptr) {
    bf16 h[4], l[4];
    split_bf16(v.x, h[0], l[0]); split_bf16(v.y, h[1], l[1]); split_bf16(v.z, h[2], l[2]); split_bf16(v.w, h[3], l[3]);
    *(uint2*)hi_ptr = *(const uint2*)h;
    *(uint2*)lo_ptr = *(const uint2*)l;
}

__global__ void __launch_bounds__(NORM_THREADS) embed_norm_kernel(const bf16* __restrict__ embed, const int* __restrict__ row_tok,
                                                                  const float* __restrict__ gain, float eps, int d,
                                                                  float* __restrict__ x, bf16* __restrict__ h_hi, bf16* __restrict__ h_lo) {
    pdl_trigger();
    pdl_wait();
    __shared__ float red[32];
    const int row = blockIdx.x, chunks = d >> 2;
    const bf16* e = embed + (size_t)row_tok[row] * d;
    float4 v[NORM_MAX_CHUNKS];
    float ss = 0.0f;
#pragma unroll
    for (int u = 0; u < NORM_MAX_CHUNKS; ++u) {
        const int c = threadIdx.x + u * NORM_THREADS;
        v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < chunks) {
            const uint2 raw = *(const uint2*)(e + 4 * c);
            const bf16* b = (const bf16*)&raw;
            v[u] = make_float4(__bfloat162float(b[0]), __bfloat162float(b[1]), __bfloat162float(b[2]), __bfloat162float(b[3]));
            *(float4*)(x + (size_t)row * d + 4 * c) = v[u];
            ss += v[u].x * v[u].x + v[u].y * v[u].y + v[u].z * v[u].z + v[u].w * v[u].w;
        }
    }
    const float rstd = rsqrtf(block_sum_1024(ss, red) / (float)d + eps);
#pragma unroll
    for (int u = 0; u < NORM_MAX_CHUNKS; ++u) {
        const int c = threadIdx.x + u * NORM_THREADS;
        if (c < chunks) {
            const float4 g = *(const float4*)(gain + 4 * c);
            store_split4(make_float4(v[u].x * rstd * g.x, v[u].y * rstd * g.y, v[u].z * rstd * g.z, v[u].w * rstd * g.w),
                         h_hi + (size_t)row * d + 4 * c, h_lo + (size_t)row * d + 4 * c);
        }
    }
}

// Single-sequence steps (row-range projections): x = E[tok]; the first projection's operand image receives
// x * gain as hi + lo terms, un-normalised; the row's sum of squares goes to ss[0][row] (one partial).
__global__ void __launch_bounds__(NORM_THREADS) embed_img_kernel(const bf16* __restrict__ embed, const int* __restrict__ row_tok,
                                                                 const float* __restrict__ gain, int d, float* __restrict__ x,
                                                                 unsigned char* __restrict__ img, float* __restrict__ ss) {
    pdl_trigger();
    pdl_wait();
    __shared__ float red[32];
    const int row = blockIdx.x, chunks = d >> 2;
    const bf16* e = embed + (size_t)row_tok[row] * d;
    float acc = 0.0f;
    for (int c = threadIdx.x; c < chunks; c += NORM_THREADS) {
        const uint2 raw = *(const uint2*)(e + 4 * c);
        const bf16* b = (const bf16*)&raw;
        const float4 g = *(const float4*)(gain + 4 * c);
        const float v[4] = {__bfloat162float(b[0]), __bfloat162float(b[1]), __bfloat162float(b[2]), __bfloat162float(b[3])};
        const float gg[4] = {g.x, g.y, g.z, g.w};
        *(float4*)(x + (size_t)row * d + 4 * c) = make_float4(v[0], v[1], v[2], v[3]);
        bf16 hi[4], lo[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) { split_bf16(v[t] * gg[t], hi[t], lo[t]); acc += v[t] * v[t]; }
        *(uint2*)(img + act_img_offset(row, 4 * c)) = *(const uint2*)hi;               // 4 elements never straddle a 16-byte chunk
        *(uint2*)(img + act_img_offset(ANPD_ROWS + row, 4 * c)) = *(const uint2*)lo;
    }
    const float t = block_sum_1024(acc, red);
    if (threadIdx.x == 0) ss[row] = t;
}

// x[row] += sum of the tile's partial sums (in segment order); then h = rmsnorm(x) * gain as hi + lo.
__global__ void __launch_bounds__(NORM_THREADS) resid_norm_kernel(float* __restrict__ x, const float* __restrict__ part,
                                                                  const int* __restrict__ seg_count, size_t split_stride, int ld_part,
                                                                  const float* __restrict__ gain, float eps, int d,
                                                                  bf16* __restrict__ h_hi, bf16* __restrict__ h_lo, int ns_max) {
    // ns_max: the most partial sums any tile of this projection has.  The loads cover that many slabs whatever the tile's own
    // count (slabs beyond it hold older sums: read, never added), so they do not wait for the count to arrive.
    pdl_trigger();
    __shared__ float red[32];
    const int row = blockIdx.x, chunks = d >> 2;
    float4 v[NORM_MAX_CHUNKS], gn[NORM_MAX_CHUNKS];
    // the norm's gain is a weight: nothing of this step writes it, so it is fetched before the dependency wait
#pragma unroll
    for (int u = 0; u < NORM_MAX_CHUNKS; ++u) {
        const int c = threadIdx.x + u * NORM_THREADS;
        gn[u] = (c < chunks) ? *(const float4*)(gain + 4 * c) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    pdl_wait();
    float ss = 0.0f;
#pragma unroll
    for (int u = 0; u < NORM_MAX_CHUNKS; ++u) {
        const int c = threadIdx.x + u * NORM_THREADS;
        v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < chunks) {
            const int ns = seg_count[(4 * c) >> 7];
            const float* pr = part + (size_t)row * ld_part + 4 * c;
            float4 acc = *(const float4*)(x + (size_t)row * d + 4 * c);
            for (int s0 = 0; s0 < ns_max; s0 += 8) {
                float4 p[8];
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    p[k] = (s0 + k < ns_max) ? *(const float4*)(pr + (size_t)(s0 + k) * split_stride) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if (s0 + k < ns) { acc.x += p[k].x; acc.y += p[k].y; acc.z += p[k].z; acc.w += p[k].w; }
            }
            v[u] = acc;
            *(float4*)(x + (size_t)row * d + 4 * c) = acc;
            ss += acc.x * acc.x + acc.y * acc.y + acc.z * acc.z + acc.w * acc.w;
        }
    }
    const float rstd = rsqrtf(block_sum_1024(ss, red) / (float)d + eps);
#pragma unroll
    for (int u = 0; u < NORM_MAX_CHUNKS; ++u) {
        const int c = threadIdx.x + u * NORM_THREADS;
        if (c < chunks) {
            const float4 g = gn[u];
            store_split4(make_float4(v[u].x * rstd * g.x, v[u].y * rstd * g.y, v[u].z * rstd * g.z, v[u].w * rstd * g.w),
                         h_hi + (size_t)row * d + 4 * c, h_lo + (size_t)row * d + 4 * c);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// QKV epilogue: reduce splits, rotary embedding, append K/V to the paged cache, keep q
// ---------------------------------------------------------------------------------------------
__global__ void qkv_rope_append_kernel(const float* __restrict__ part, const int* __restrict__ seg_count, size_t split_stride, int ld_part,
                                       const int* __restrict__ row_pos, const int* __restrict__ row_slot, const int* __restrict__ row_seq,
                                       const int* __restrict__ row_ok, const float* __restrict__ rope_cos,
                                       const float* __restrict__ rope_sin, const int* __restrict__ page_table,
                                       int pages_per_seq, int Hq, int Hkv, int hd, float q_scale, bf16* __restrict__ q_hi,
                                       bf16* __restrict__ q_lo, bf16* __restrict__ kpool_l, bf16* __restrict__ vpool_l, int ns_max) {
    pdl_trigger();
    pdl_wait();
    // a block covers blockDim.x / (hd / 2) consecutive heads of one row
    const int half = hd >> 1, row = blockIdx.x, head = blockIdx.y * (blockDim.x / half) + threadIdx.x / half, i = threadIdx.x % half;
    if (head >= Hq + 2 * Hkv) return;
    const float* pr = part + (size_t)row * ld_part + (size_t)head * hd;
    float a = 0.0f, b = 0.0f;
    // up to four slabs are requested before the tile's own count is known (ns_max: the projection's largest count)
    float pa[4], pb[4];
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        pa[s] = (s < ns_max) ? pr[s * split_stride + i] : 0.0f;
        pb[s] = (s < ns_max) ? pr[s * split_stride + i + half] : 0.0f;
    }
    const int ns = seg_count[(head * hd + i) >> 7];      // a head never straddles a 128-column tile
    const int pos = row_pos[row];
#pragma unroll
    for (int s = 0; s < 4; ++s) if (s < ns) { a += pa[s]; b += pb[s]; }
    for (int s = 4; s < ns; ++s) { a += pr[s * split_stride + i]; b += pr[s * split_stride + i + half]; }
    if (head < Hq + Hkv) {
        const float c = rope_cos[(size_t)pos * half + i], sn = rope_sin[(size_t)pos * half + i];
        const float ra = a * c - b * sn, rb = b * c + a * sn;
        a = ra; b = rb;
    }
    if (head < Hq) {
        // queries leave as two bf16 terms, already multiplied by log2(e) / sqrt(hd): the attention kernel
        // takes them as MMA fragments and works with base-2 exponentials
        const size_t o = (size_t)row * Hq * hd + head * hd + i;
        split_bf16(a * q_scale, q_hi[o], q_lo[o]);
        split_bf16(b * q_scale, q_hi[o + half], q_lo[o + half]);
        return;
    }
    if (!row_ok[row]) return;
    const bool is_k = head < Hq + Hkv;
    const int kvh = is_k ? head - Hq : head - Hq - Hkv;
    const int slot = row_slot[row];               // where the row lives in the cache (its position, except for a second candidate)
    const int page = page_table[row_seq[row] * pages_per_seq + slot / KV_PAGE];
    bf16* pg = (is_k ? kpool_l : vpool_l) + ((size_t)page * Hkv + kvh) * KV_PAGE * hd;
    if (is_k) {                                   // K page: [position][dim]
        pg[(size_t)(slot % KV_PAGE) * hd + i] = __float2bfloat16_rn(a);
        pg[(size_t)(slot % KV_PAGE) * hd + i + half] = __float2bfloat16_rn(b);
    } else {                                      // V page is kept transposed: [dim][position]
        pg[(size_t)i * KV_PAGE + (slot % KV_PAGE)] = __float2bfloat16_rn(a);
        pg[(size_t)(i + half) * KV_PAGE + (slot % KV_PAGE)] = __float2bfloat16_rn(b);
    }
}

// The same for a prompt pass (rows are consecutive positions of one sequence, a multiple of 8, the first a multiple of 64):
// a block takes 64 rows of one head through shared memory, so that the transposed V page receives whole 16-byte runs of
// positions instead of single elements.  Per element the arithmetic is that of qkv_rope_append_kernel, in the same order.
constexpr int ROPE_TILE_ROWS = 64;
template <int HD>
__global__ void __launch_bounds__(256) qkv_rope_append_tile_kernel(const float* __restrict__ part, const int* __restrict__ seg_count, size_t split_stride,
                                                                   int ld_part, int rows, const int* __restrict__ row_pos, const int* __restrict__ row_seq,
                                                                   const int* __restrict__ row_ok, const float* __restrict__ rope_cos,
                                                                   const float* __restrict__ rope_sin, const int* __restrict__ page_table,
                                                                   int pages_per_seq, int Hq, int Hkv, float q_scale, bf16* __restrict__ q_hi,
                                                                   bf16* __restrict__ q_lo, bf16* __restrict__ kpool_l, bf16* __restrict__ vpool_l) {
    pdl_trigger();
    pdl_wait();
    __shared__ float tile[ROPE_TILE_ROWS][HD + 1];
    constexpr int half = HD / 2;
    const int r0 = blockIdx.x * ROPE_TILE_ROWS, head = blockIdx.y;
    const int nr = min(ROPE_TILE_ROWS, rows - r0);
    const int ns = seg_count[(head * HD) >> 7];          // a head never straddles a 128-column tile
    // 16-byte loads, eight of them in flight per thread
    constexpr int Q4 = HD / 4;
    for (int base = 0; base < nr * Q4; base += 8 * 256) {
        float4 a[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {                     // the first partial sums (there is always one): eight independent loads
            const int idx = base + u * 256 + threadIdx.x;
            a[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (idx < nr * Q4) a[u] = *(const float4*)(part + (size_t)(r0 + idx / Q4) * ld_part + (size_t)head * HD + (idx % Q4) * 4);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int idx = base + u * 256 + threadIdx.x;
            if (idx >= nr * Q4) continue;
            const int r = idx / Q4, dim = (idx % Q4) * 4;
            const float* pr = part + (size_t)(r0 + r) * ld_part + (size_t)head * HD + dim;
            for (int s = 1; s < ns; ++s) { const float4 v = *(const float4*)(pr + s * split_stride); a[u].x += v.x; a[u].y += v.y; a[u].z += v.z; a[u].w += v.w; }
            tile[r][dim] = a[u].x; tile[r][dim + 1] = a[u].y; tile[r][dim + 2] = a[u].z; tile[r][dim + 3] = a[u].w;
        }
    }
    __syncthreads();
    if (head < Hq + Hkv) {
        for (int idx = threadIdx.x; idx < nr * half; idx += 256) {
            const int r = idx / half, i = idx % half;
            const int pos = row_pos[r0 + r];
            const float a = tile[r][i], b = tile[r][i + half];
            const float c = rope_cos[(size_t)pos * half + i], sn = rope_sin[(size_t)pos * half + i];
            tile[r][i] = a * c - b * sn;
            tile[r][i + half] = b * c + a * sn;
        }
        __syncthreads();
    }
    if (head < Hq) {
        for (int idx = threadIdx.x; idx < nr * Q4; idx += 256) {
            const int r = idx / Q4, dim = (idx % Q4) * 4;
            const size_t o = (size_t)(r0 + r) * Hq * HD + (size_t)head * HD + dim;
            store_split4(make_float4(tile[r][dim] * q_scale, tile[r][dim + 1] * q_scale, tile[r][dim + 2] * q_scale, tile[r][dim + 3] * q_scale),
                         q_hi + o, q_lo + o);
        }
        return;
    }
    const bool is_k = head < Hq + Hkv;
    const int kvh = is_k ? head - Hq : head - Hq - Hkv;
    const int pos0 = row_pos[r0];                        // the tile's rows hold positions pos0, pos0 + 1, ... inside one page
    const int page = page_table[row_seq[r0] * pages_per_seq + pos0 / KV_PAGE];
    bf16* pg = (is_k ? kpool_l : vpool_l) + ((size_t)page * Hkv + kvh) * KV_PAGE * HD;
    if (is_k) {                                          // K page: [position][dim]
        for (int idx = threadIdx.x; idx < nr * Q4; idx += 256) {
            const int r = idx / Q4, dim = (idx % Q4) * 4;
            if (!row_ok[r0 + r]) continue;
            bf16 v[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) v[e] = __float2bfloat16_rn(tile[r][dim + e]);
            *(uint2*)(pg + (size_t)((pos0 + r) % KV_PAGE) * HD + dim) = *(const uint2*)v;
        }
    } else {                                             // V page, transposed: [dim][position]; 8 positions = 16 bytes
        for (int idx = threadIdx.x; idx < (ROPE_TILE_ROWS / 8) * HD; idx += 256) {
            const int dim = idx % HD, r8 = (idx / HD) * 8;
            if (r8 >= nr) continue;
            bf16 v[8];
            bool all = true;
#pragma unroll
            for (int e = 0; e < 8; ++e) { v[e] = __float2bfloat16_rn(tile[r8 + e][dim]); all = all && row_ok[r0 + r8 + e] != 0; }
            bf16* dst = pg + (size_t)dim * KV_PAGE + (pos0 % KV_PAGE) + r8;
            if (all) *(uint4*)dst = *(const uint4*)v;
            else
                for (int e = 0; e < 8; ++e) if (row_ok[r0 + r8 + e]) dst[e] = v[e];
        }
    }
}

// ---------------------------------------------------------------------------------------------
// attention: per (key page, kv head, group of 8 rows) partial softmax, then a combine in page order
//
// The partial kernel works on tensor cores (mma.sync m16n8k16, bf16 in, fp32 out).  A K page is
// [128 keys][hd] and a V page is stored transposed, [hd][128 keys], so both are the "column" operand
// of an MMA and each thread fetches 16 contiguous bytes per fragment.  A block first issues every
// 16-byte asynchronous copy of its K and V page into (row-padded, bank-conflict-free) shared memory,
// so one block keeps up to 64 KB in flight, then computes from shared memory.  The
// 8 rows x G query heads that share a kv head are the MMA's 16-row tiles.  q and the softmax weights
// enter as two bf16 terms each (hi + lo), so only the cache's own bf16 rounding is left.  A warp walks
// its 32-key blocks in position order with a running (max, sum, output); warps that split a page are
// merged in block order; pages are merged by the combine kernel in page order.  Every one of these
// orders is a function of absolute key positions only, and a masked key contributes an exact zero,
// so a row's result does not depend on which other rows share the launch.
//
// Fragment bookkeeping (g = lane / 4, t = lane % 4): a 16-byte load gives a thread 8 consecutive
// elements e0..e7 of the contraction dimension; (e0,e1),(e2,e3) feed one MMA and (e4,e5),(e6,e7) a
// second one, and the other operand is permuted the same way, which leaves the sum unchanged.  For
// QK^T the key a thread column maps to is chosen so that the score fragments are, as they stand,
// the P fragments the PV product needs: logical key 8j + 2t + e of a block is actual key 8t + 2j + e.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void mma_bf16_16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// (x, y) -> packed bf16 pair of the high parts; `lo` receives the packed pair of the remainders.
__device__ __forceinline__ uint32_t pack_split(float x, float y, uint32_t& lo) {
    const bf16 hx = __float2bfloat16_rn(x), hy = __float2bfloat16_rn(y);
    const bf16 lx = __float2bfloat16_rn(x - __bfloat162float(hx)), ly = __float2bfloat16_rn(y - __bfloat162float(hy));
    lo = (uint32_t)__bfloat16_as_ushort(lx) | ((uint32_t)__bfloat16_as_ushort(ly) << 16);
    return (uint32_t)__bfloat16_as_ushort(hx) | ((uint32_t)__bfloat16_as_ushort(hy) << 16);
}

constexpr int ATTN_THREADS = 128;
constexpr int KEY_BLOCK = 32;

template <int HD>
__global__ void __launch_bounds__(ATTN_THREADS) attn_partial_kernel(const bf16* __restrict__ q_hi, const bf16* __restrict__ q_lo,
                                                                    const bf16* __restrict__ kpool_l, const bf16* __restrict__ vtpool_l,
                                                                    const int* __restrict__ page_table, int pages_per_seq,
                                                                    const int* __restrict__ row_pos, const int* __restrict__ row_seq, int Hq,
                                                                    int Hkv, float* __restrict__ pm, float* __restrict__ pl,
                                                                    float* __restrict__ po, const int* __restrict__ row_slot,
                                                                    const int* __restrict__ row_hole_lo, const int* __restrict__ row_hole_hi) {
    pdl_trigger();
    pdl_wait();
    constexpr int SLABS = HD / 32;            // 32-wide slabs of the head dimension (two MMAs each)
    constexpr int DT = HD / 8;                // 8-wide tiles of the head dimension for P V
    constexpr int OP = HD + 4;                // padded row of the merge buffer
    constexpr int KPITCH = HD * 2 + 64;       // bytes per staged K row (64 bytes of padding: conflict-free 16-byte reads)
    constexpr int VPITCH = KV_PAGE * 2 + 64;  // bytes per staged V^T row
    extern __shared__ __align__(16) unsigned char attn_smem[];
    unsigned char* Ks = attn_smem;                                  // [KV_PAGE][KPITCH]
    unsigned char* Vs = attn_smem + KV_PAGE * KPITCH;               // [HD][VPITCH]
    float (*sm_o)[16][OP] = (float (*)[16][OP])Ks;                  // [4][16][OP], reuses the K staging area after the last MMA
    __shared__ float sm_m[4][16], sm_l[4][16], sm_w[4][16];

    const int G = Hq / Hkv;
    const int MT = (ANPD_ROWS * G + 15) / 16;             // 16-row tiles of query vectors: 1, 1, 2, 4 for G = 1, 2, 4, 8
    const int KG = 4 / MT;                                // warps that split the page's four key blocks
    const int c = blockIdx.x, kvh = blockIdx.y, r0 = blockIdx.z * ANPD_ROWS;
    // row_slot (two-candidate steps): a row sees the cache slots up to its own, except a hidden range; otherwise slot = position
    const int pos_lo = row_pos[r0], pos_hi = row_slot ? row_slot[r0 + ANPD_ROWS - 1] : row_pos[r0 + ANPD_ROWS - 1];
    if (c * KV_PAGE > pos_hi) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gid = lane >> 2, t = lane & 3;
    const int mt = warp % MT, kg = warp / MT;
    const int page = page_table[row_seq[r0] * pages_per_seq + c];
    const bf16* Kg = kpool_l + ((size_t)page * Hkv + kvh) * KV_PAGE * HD;
    const bf16* Vg = vtpool_l + ((size_t)page * Hkv + kvh) * KV_PAGE * HD;

    // stage the part of the page that any row can see: whole 32-key blocks up to pos_hi
    {
        const int nblk = min(KV_PAGE / KEY_BLOCK, (pos_hi - c * KV_PAGE) / KEY_BLOCK + 1);
        constexpr int KCH = HD * 2 / 16;                  // 16-byte chunks per K row
        for (int i = threadIdx.x; i < nblk * KEY_BLOCK * KCH; i += ATTN_THREADS) {
            const int row = i / KCH, ch = i % KCH;
            const uint32_t dst = (uint32_t)__cvta_generic_to_shared(Ks + row * KPITCH + ch * 16);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(Kg + (size_t)row * HD + ch * 8) : "memory");
        }
        const int vch = nblk * (KEY_BLOCK * 2 / 16);      // chunks per V^T row that hold visible keys
        for (int i = threadIdx.x; i < HD * vch; i += ATTN_THREADS) {
            const int row = i / vch, ch = i % vch;
            const uint32_t dst = (uint32_t)__cvta_generic_to_shared(Vs + row * VPITCH + ch * 16);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(Vg + (size_t)row * KV_PAGE + ch * 8) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    }

    // this thread's two query vectors (rows gid and gid + 8 of tile mt) and their positions
    int qpos[2], qhl[2] = {0, 0}, qhh[2] = {0, 0};
    uint32_t qh[SLABS][2][4], ql[SLABS][2][4];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int qi = mt * 16 + gid + 8 * h;
        const bool valid = qi < ANPD_ROWS * G;
        const int r = valid ? qi / G : 0, hl = valid ? qi % G : 0;
        qpos[h] = valid ? (row_slot ? row_slot[r0 + r] : pos_lo + r) : -1;                // -1: padding row, sees no key
        if (valid && row_slot) { qhl[h] = row_hole_lo[r0 + r]; qhh[h] = row_hole_hi[r0 + r]; }
        const size_t qoff = (size_t)(r0 + r) * Hq * HD + (size_t)(kvh * G + hl) * HD + 8 * t;
#pragma unroll
        for (int s = 0; s < SLABS; ++s) {
            // 16 bytes = elements 8t..8t+7 of the slab: (e0,e1),(e2,e3) feed the slab's first MMA, (e4,e5),(e6,e7)
            // the second.  Register h holds row gid + 8h for logical k = 2t, 2t+1; register 2 + h for 2t+8, 2t+9.
            uint4 a = make_uint4(0u, 0u, 0u, 0u), b = a;
            if (valid) { a = *(const uint4*)(q_hi + qoff + 32 * s); b = *(const uint4*)(q_lo + qoff + 32 * s); }
            qh[s][0][h] = a.x; qh[s][0][2 + h] = a.y; qh[s][1][h] = a.z; qh[s][1][2 + h] = a.w;
            ql[s][0][h] = b.x; ql[s][0][2 + h] = b.y; ql[s][1][h] = b.z; ql[s][1][2 + h] = b.w;
        }
    }

    float m_run[2] = {-CUDART_INF_F, -CUDART_INF_F}, l_run[2] = {0.f, 0.f};
    float o[DT][4];
#pragma unroll
    for (int d = 0; d < DT; ++d) { o[d][0] = 0.f; o[d][1] = 0.f; o[d][2] = 0.f; o[d][3] = 0.f; }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();

    for (int blk = kg; blk < KV_PAGE / KEY_BLOCK; blk += KG) {
        const int kb0 = c * KV_PAGE + blk * KEY_BLOCK;
        if (kb0 > pos_hi) break;
        // ---- scores of 16 query vectors x 32 keys ----
        float sc[4][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            sc[j][0] = 0.f; sc[j][1] = 0.f; sc[j][2] = 0.f; sc[j][3] = 0.f;
            const int key_local = blk * KEY_BLOCK + 8 * (gid >> 1) + 2 * j + (gid & 1);
            const unsigned char* kr = Ks + key_local * KPITCH + 16 * t;
#pragma unroll
            for (int s = 0; s < SLABS; ++s) {
                const uint4 kv = *(const uint4*)(kr + 64 * s);
                mma_bf16_16816(sc[j], qh[s][0], kv.x, kv.y);
                mma_bf16_16816(sc[j], ql[s][0], kv.x, kv.y);
                mma_bf16_16816(sc[j], qh[s][1], kv.z, kv.w);
                mma_bf16_16816(sc[j], ql[s][1], kv.z, kv.w);
            }
        }
        // ---- running softmax per row; sc[j][2h + e] belongs to row h, actual key kb0 + 8t + 2j + e ----
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float mx = -CUDART_INF_F;
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int key = kb0 + 8 * t + 2 * j + e;
                    const float v = (key <= qpos[h] && !(key >= qhl[h] && key < qhh[h])) ? sc[j][2 * h + e] : -CUDART_INF_F;
                    sc[j][2 * h + e] = v;
                    mx = fmaxf(mx, v);
                }
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m_run[h], mx);
            const bool none = (m_new == -CUDART_INF_F);
            const float resc = none ? 1.0f : exp2f(m_run[h] - m_new);
            float psum = 0.0f;
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const float p = none ? 0.0f : exp2f(sc[j][2 * h + e] - m_new);
                    sc[j][2 * h + e] = p;
                    psum += p;
                }
            psum += __shfl_xor_sync(0xffffffffu, psum, 1);
            psum += __shfl_xor_sync(0xffffffffu, psum, 2);
            l_run[h] = l_run[h] * resc + psum;
            m_run[h] = m_new;
#pragma unroll
            for (int d = 0; d < DT; ++d) { o[d][2 * h] *= resc; o[d][2 * h + 1] *= resc; }
        }
        // ---- P fragments (hi + lo) for the two MMAs over this block's 32 keys ----
        uint32_t ph[2][4], plo[2][4];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            ph[u][0] = pack_split(sc[2 * u][0], sc[2 * u][1], plo[u][0]);            // row gid,     keys 8t + 4u + {0,1}
            ph[u][1] = pack_split(sc[2 * u][2], sc[2 * u][3], plo[u][1]);            // row gid + 8
            ph[u][2] = pack_split(sc[2 * u + 1][0], sc[2 * u + 1][1], plo[u][2]);    // row gid,     keys 8t + 4u + {2,3}
            ph[u][3] = pack_split(sc[2 * u + 1][2], sc[2 * u + 1][3], plo[u][3]);    // row gid + 8
        }
        // ---- O += P V : V^T rows are head dimensions, 16 bytes = keys 8t .. 8t+7 of the block ----
#pragma unroll
        for (int d = 0; d < DT; ++d) {
            const uint4 vv = *(const uint4*)(Vs + (8 * d + gid) * VPITCH + (blk * KEY_BLOCK + 8 * t) * 2);
            mma_bf16_16816(o[d], ph[0], vv.x, vv.y);
            mma_bf16_16816(o[d], plo[0], vv.x, vv.y);
            mma_bf16_16816(o[d], ph[1], vv.z, vv.w);
            mma_bf16_16816(o[d], plo[1], vv.z, vv.w);
        }
    }

    // ---- merge the warps that split this page (block order), write the page's partial ----
    __syncthreads();                                      // every warp is done reading the staged K rows
    if (t == 0) {
        sm_m[warp][gid] = m_run[0]; sm_m[warp][gid + 8] = m_run[1];
        sm_l[warp][gid] = l_run[0]; sm_l[warp][gid + 8] = l_run[1];
    }
#pragma unroll
    for (int d = 0; d < DT; ++d) {
        sm_o[warp][gid][8 * d + 2 * t] = o[d][0];
        sm_o[warp][gid][8 * d + 2 * t + 1] = o[d][1];
        sm_o[warp][gid + 8][8 * d + 2 * t] = o[d][2];
        sm_o[warp][gid + 8][8 * d + 2 * t + 1] = o[d][3];
    }
    __syncthreads();
    // weights of the merged warps, once per query vector
    if (threadIdx.x < MT * 16) {
        const int tile = threadIdx.x / 16, rowi = threadIdx.x % 16;
        float M = -CUDART_INF_F;
        for (int k = 0; k < KG; ++k) M = fmaxf(M, sm_m[k * MT + tile][rowi]);
        float L = 0.0f;
        for (int k = 0; k < KG; ++k) {
            const float mk = sm_m[k * MT + tile][rowi];
            const float w = (mk == -CUDART_INF_F) ? 0.0f : exp2f(mk - M);
            sm_w[k * MT + tile][rowi] = w;
            L = fmaf(sm_l[k * MT + tile][rowi], w, L);
        }
        const int qi = tile * 16 + rowi;
        if (qi < ANPD_ROWS * G) {
            const size_t out = ((size_t)(r0 + qi / G) * Hq + (kvh * G + qi % G)) * pages_per_seq + c;
            pm[out] = M;
            pl[out] = L;
        }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < MT * 16 * (HD / 4); idx += ATTN_THREADS) {
        const int d4 = idx % (HD / 4), rowi = (idx / (HD / 4)) % 16, tile = idx / ((HD / 4) * 16);
        const int qi = tile * 16 + rowi;
        if (qi >= ANPD_ROWS * G) continue;
        float4 O = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int k = 0; k < KG; ++k) {
            const float w = sm_w[k * MT + tile][rowi];
            const float4 v = *(const float4*)&sm_o[k * MT + tile][rowi][4 * d4];
            O.x = fmaf(v.x, w, O.x); O.y = fmaf(v.y, w, O.y); O.z = fmaf(v.z, w, O.z); O.w = fmaf(v.w, w, O.w);
        }
        const size_t out = ((size_t)(r0 + qi / G) * Hq + (kvh * G + qi % G)) * pages_per_seq + c;
        *(float4*)(po + out * HD + 4 * d4) = O;
    }
}

// One block per (row, q head): fold the pages 0..pos/KV_PAGE, write the output as hi+lo.  The block is
// hd x 4 threads: thread (dim, k) adds the pages k, k+4, k+8, ... in ascending order, the four slices
// are then added in slice order - a fixed order for a given number of pages.  Page maxima and sums are
// fetched once by the first threads, so the kernel is about two memory round trips long.
constexpr int COMBINE_SLICES = 4;
constexpr int COMBINE_MAX_PAGES = 256;
__global__ void attn_combine_kernel(const float* __restrict__ pm, const float* __restrict__ pl, const float* __restrict__ po,
                                    const int* __restrict__ row_pos, int Hq, int hd, int pages_per_seq,
                                    bf16* __restrict__ ao_hi, bf16* __restrict__ ao_lo, unsigned char* __restrict__ img) {
    // row_pos: the rows' cache slots (= positions outside two-candidate steps)
    pdl_trigger();
    pdl_wait();
    __shared__ float s_w[COMBINE_MAX_PAGES];            // page maxima, then page weights
    __shared__ float s_l[COMBINE_MAX_PAGES];
    __shared__ float s_o[COMBINE_SLICES][128];
    __shared__ float s_L;
    const int row = blockIdx.x, head = blockIdx.y;
    const int dim = threadIdx.x % hd, slice = threadIdx.x / hd;
    const int nc = min(row_pos[row] / KV_PAGE + 1, COMBINE_MAX_PAGES);
    const size_t base = ((size_t)row * Hq + head) * pages_per_seq;
    for (int c = threadIdx.x; c < nc; c += blockDim.x) { s_w[c] = pm[base + c]; s_l[c] = pl[base + c]; }
    __syncthreads();
    float M = -CUDART_INF_F;
    for (int c = 0; c < nc; ++c) M = fmaxf(M, s_w[c]);
    __syncthreads();
    for (int c = threadIdx.x; c < nc; c += blockDim.x) s_w[c] = exp2f(s_w[c] - M);     // partial maxima are in the base-2 domain
    __syncthreads();
    if (threadIdx.x == 0) {
        float L = 0.0f;
        for (int c = 0; c < nc; ++c) L = fmaf(s_l[c], s_w[c], L);
        s_L = L;
    }
    float o = 0.0f;
    for (int c0 = slice; c0 < nc; c0 += 4 * COMBINE_SLICES) {
        float v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int c = c0 + u * COMBINE_SLICES;
            v[u] = (c < nc) ? po[(base + c) * hd + dim] : 0.0f;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int c = c0 + u * COMBINE_SLICES;
            if (c < nc) o = fmaf(v[u], s_w[c], o);
        }
    }
    s_o[slice][dim] = o;
    __syncthreads();
    if (slice == 0) {
        float t = s_o[0][dim];
        for (int k = 1; k < COMBINE_SLICES; ++k) t += s_o[k][dim];
        bf16 hi, lo;
        split_bf16(t / s_L, hi, lo);
        if (img) {                                        // single-sequence step: straight into the O projection's operand image
            *(bf16*)(img + act_img_offset(row, head * hd + dim)) = hi;
            *(bf16*)(img + act_img_offset(ANPD_ROWS + row, head * hd + dim)) = lo;
        } else {
            const size_t out = (size_t)row * Hq * hd + head * hd + dim;
            ao_hi[out] = hi;
            ao_lo[out] = lo;
        }
    }
}

// The same for many rows (prefill passes), shaped for throughput: four warps per (row, q head), a lane owns hd/32
// consecutive dimensions and fetches them in one load per page.  Slices, page order within a slice, the order of the
// slices and the total weight are those of attn_combine_kernel, so the results are the same bits.
template <int VEC>
__global__ void __launch_bounds__(32 * COMBINE_SLICES) attn_combine_wide_kernel(const float* __restrict__ pm, const float* __restrict__ pl,
                                                                               const float* __restrict__ po, const int* __restrict__ row_pos,
                                                                               int Hq, int pages_per_seq, bf16* __restrict__ ao_hi,
                                                                               bf16* __restrict__ ao_lo) {
    pdl_trigger();
    pdl_wait();
    constexpr int hd = 32 * VEC;
    __shared__ float s_m[COMBINE_MAX_PAGES];
    __shared__ float s_l[COMBINE_MAX_PAGES];
    __shared__ float s_o[COMBINE_SLICES][hd];
    const int row = blockIdx.x, head = blockIdx.y;
    const int lane = threadIdx.x & 31, slice = threadIdx.x >> 5;
    const int nc = min(row_pos[row] / KV_PAGE + 1, COMBINE_MAX_PAGES);
    const size_t base = ((size_t)row * Hq + head) * pages_per_seq;
    for (int c = threadIdx.x; c < nc; c += blockDim.x) { s_m[c] = pm[base + c]; s_l[c] = pl[base + c]; }
    __syncthreads();
    float M = -CUDART_INF_F;
    for (int c = 0; c < nc; ++c) M = fmaxf(M, s_m[c]);
    float L = 0.0f;
    for (int c = 0; c < nc; ++c) L = fmaf(s_l[c], exp2f(s_m[c] - M), L);       // partial maxima are in the base-2 domain
    float o[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) o[e] = 0.0f;
    for (int c = slice; c < nc; c += COMBINE_SLICES) {
        const float w = exp2f(s_m[c] - M);
        const float* src = po + (base + c) * hd + lane * VEC;
        float v[VEC];
        if (VEC == 4) { const float4 t = *(const float4*)src; v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
        else { const float2 t = *(const float2*)src; v[0] = t.x; v[1] = t.y; }
#pragma unroll
        for (int e = 0; e < VEC; ++e) o[e] = fmaf(v[e], w, o[e]);
    }
#pragma unroll
    for (int e = 0; e < VEC; ++e) s_o[slice][lane * VEC + e] = o[e];
    __syncthreads();
    if (slice == 0) {
        const size_t out = (size_t)row * Hq * hd + head * hd + lane * VEC;
        bf16 h[VEC], l[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            float t = s_o[0][lane * VEC + e];
            for (int k = 1; k < COMBINE_SLICES; ++k) t += s_o[k][lane * VEC + e];
            split_bf16(t / L, h[e], l[e]);
        }
        if (VEC == 4) { *(uint2*)(ao_hi + out) = *(const uint2*)h; *(uint2*)(ao_lo + out) = *(const uint2*)l; }
        else { *(uint32_t*)(ao_hi + out) = *(const uint32_t*)h; *(uint32_t*)(ao_lo + out) = *(const uint32_t*)l; }
    }
}

// ---------------------------------------------------------------------------------------------
// SwiGLU epilogue of the gate/up projection
// ---------------------------------------------------------------------------------------------
__global__ void swiglu_kernel(const float* __restrict__ part, const int* __restrict__ seg_count, size_t split_stride, int ld_part, int F,
                              bf16* __restrict__ act_hi, bf16* __restrict__ act_lo, int ns_max) {
    pdl_trigger();
    pdl_wait();
    const int row = blockIdx.y, j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= F) return;
    const float* pr = part + (size_t)row * ld_part;
    float gte = 0.0f, up = 0.0f;
    // up to four slabs are requested before the tile's own count is known (ns_max: the projection's largest count)
    float pg[4], pu[4];
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        pg[s] = (s < ns_max) ? pr[s * split_stride + j] : 0.0f;
        pu[s] = (s < ns_max) ? pr[s * split_stride + F + j] : 0.0f;
    }
    const int ng = seg_count[j >> 7], nu = seg_count[(F + j) >> 7];
#pragma unroll
    for (int s = 0; s < 4; ++s) { if (s < ng) gte += pg[s]; if (s < nu) up += pu[s]; }
    for (int s = 4; s < ng; ++s) gte += pr[s * split_stride + j];
    for (int s = 4; s < nu; ++s) up += pr[s * split_stride + F + j];
    const float v = gte / (1.0f + expf(-gte)) * up;
    bf16 hi, lo;
    split_bf16(v, hi, lo);
    act_hi[(size_t)row * F + j] = hi;
    act_lo[(size_t)row * F + j] = lo;
}

// The same for many rows (prefill passes): a thread owns four consecutive features, so the partial sums come in
// 16-byte loads.  Per element the arithmetic is that of swiglu_kernel, in the same order.
__global__ void swiglu_wide_kernel(const float* __restrict__ part, const int* __restrict__ seg_count, size_t split_stride, int ld_part, int F,
                                   bf16* __restrict__ act_hi, bf16* __restrict__ act_lo) {
    pdl_trigger();
    pdl_wait();
    // two chunks of four features per thread (a block's width apart); every output has at least one partial sum, so the
    // first partial sums of gate and up of both chunks are requested together, before anything depends on them
    const int row = blockIdx.y, j0 = 4 * (2 * blockIdx.x * blockDim.x + threadIdx.x);
    const float* pr = part + (size_t)row * ld_part;
    float4 g4[2], u4[2];
    int ng[2], nu[2];
    bool live[2];
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        const int j = j0 + c * 4 * blockDim.x;
        live[c] = j < F;
        g4[c] = u4[c] = make_float4(0.f, 0.f, 0.f, 0.f);
        ng[c] = nu[c] = 0;
        if (live[c]) {
            g4[c] = *(const float4*)(pr + j);
            u4[c] = *(const float4*)(pr + F + j);
            ng[c] = seg_count[j >> 7];
            nu[c] = seg_count[(F + j) >> 7];
        }
    }
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        if (!live[c]) continue;
        const int j = j0 + c * 4 * blockDim.x;
        for (int s = 1; s < ng[c]; ++s) { const float4 p = *(const float4*)(pr + s * split_stride + j); g4[c].x += p.x; g4[c].y += p.y; g4[c].z += p.z; g4[c].w += p.w; }
        for (int s = 1; s < nu[c]; ++s) { const float4 p = *(const float4*)(pr + s * split_stride + F + j); u4[c].x += p.x; u4[c].y += p.y; u4[c].z += p.z; u4[c].w += p.w; }
        const float gte[4] = {g4[c].x, g4[c].y, g4[c].z, g4[c].w}, up[4] = {u4[c].x, u4[c].y, u4[c].z, u4[c].w};
        bf16 hi[4], lo[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) split_bf16(gte[e] / (1.0f + expf(-gte[e])) * up[e], hi[e], lo[e]);
        *(uint2*)(act_hi + (size_t)row * F + j) = *(const uint2*)hi;
        *(uint2*)(act_lo + (size_t)row * F + j) = *(const uint2*)lo;
    }
}

// ---------------------------------------------------------------------------------------------
// LM-head epilogue: reduce splits, (optionally) keep logits, per-block argmax with ties to the lowest id
// ---------------------------------------------------------------------------------------------
constexpr int AMAX_COLS = 1024;
__global__ void __launch_bounds__(256) argmax_partial_kernel(const float* __restrict__ part, const int* __restrict__ seg_count, size_t split_stride,
                                                             int ld_part, int V, float* __restrict__ logits,
                                                             float* __restrict__ amax_val, int* __restrict__ amax_idx, int nblk) {
    pdl_trigger();
    pdl_wait();
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
                                                     const NgramDev* ctxs, int seq_arg, int last_row, int prompt_len, int two) {
    pdl_trigger();
    pdl_wait();
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
    const int ka = s.draft_len;
    while (a < ka && s.draft[a] == pred[a]) ++a;
    for (int r = 0; r < ANPD_ROWS; ++r) s.pred[r] = pred[r];
    // A second candidate (rows ka+1..ka+kb): its first token is judged by row 0's prediction, token j by the prediction of
    // its own row before (row ka+j).  It is kept when its accepted prefix is strictly longer; the first candidate wins ties.
    const int kb = two ? min(s.draft2_len, ANPD_K_MAX - ka) : 0;
    const int* chosen = s.draft;
    int nxt = pred[a];
    if (two) s.move_n = 0;
    if (kb > 0 && s.draft2[0] == pred[0]) {
        int ab = 1;
        while (ab < kb && s.draft2[ab] == pred[ka + ab]) ++ab;
        if (ab > a) {
            chosen = s.draft2;
            a = ab;
            nxt = pred[ka + ab];
            if (mode == ACCEPT_COMMIT && s.active) {           // its K/V rows sit behind the first candidate's: ask for the move
                s.move_from = s.kv_len + ka + 1;
                s.move_to = s.kv_len + 1;
                s.move_n = ab;
                s.alt_wins += 1;
            }
        }
    }
    s.accepted_len = a;
    s.next_tok = nxt;
    if (mode != ACCEPT_COMMIT || !s.active) return;
    s.kv_len += a + 1;
    s.steps += 1;
    s.drafted += ka + kb;
    s.accepted += a;
    s.hist[a] += 1;
    if (ctxs) {
        const NgramDev& c = ctxs[b];
        const int T = c.state[0];
        if (T + a + 1 > c.max_ctx) { s.error = ERR_CTX_FULL; s.active = 0; return; }
        for (int i = 0; i < a; ++i) c.tokens[T + i] = chosen[i];
        c.tokens[T + a] = nxt;
        c.state[0] = T + a + 1;
        if (T + a + 1 >= s.stop_at) s.active = 0;
    }
}

// Two-candidate steps: when the second candidate won, its accepted rows' K and V move from the slots behind the first
// candidate's to the positions they belong to (SeqState::move_*).  One thread per (layer, kv head, dim) walks the rows in
// ascending order, so overlapping ranges behave like memmove.  grid (layers * kv heads, batch), hd threads.
__global__ void kv_move_kernel(const SeqState* __restrict__ seqs, const int* __restrict__ page_table, int pages_per_seq, int Hkv, int hd,
                               size_t layer_elems, bf16* __restrict__ kpool, bf16* __restrict__ vpool) {
    pdl_trigger();
    pdl_wait();
    const SeqState& s = seqs[blockIdx.y];
    const int n = s.move_n;
    if (n <= 0) return;
    const int layer = blockIdx.x / Hkv, kvh = blockIdx.x % Hkv, i = threadIdx.x;
    for (int j = 0; j < n; ++j) {
        const int from = s.move_from + j, to = s.move_to + j;
        const size_t pf = ((size_t)page_table[blockIdx.y * pages_per_seq + from / KV_PAGE] * Hkv + kvh) * KV_PAGE * hd + layer * layer_elems;
        const size_t pt = ((size_t)page_table[blockIdx.y * pages_per_seq + to / KV_PAGE] * Hkv + kvh) * KV_PAGE * hd + layer * layer_elems;
        kpool[pt + (size_t)(to % KV_PAGE) * hd + i] = kpool[pf + (size_t)(from % KV_PAGE) * hd + i];
        vpool[pt + (size_t)i * KV_PAGE + (to % KV_PAGE)] = vpool[pf + (size_t)i * KV_PAGE + (from % KV_PAGE)];
    }
}

// ---------------------------------------------------------------------------------------------
// weight-streaming GEMM, plain version: one warp per output feature, 8 rows at a time
//   part[0][row][n] = sum_k W[n][k] * (a_hi[row][k] + a_lo[row][k])
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) gemm_rows8_kernel(const bf16* __restrict__ W, const bf16* __restrict__ a_hi,
                                                         const bf16* __restrict__ a_lo, int rows, int N, int K, long long total, int G,
                                                         float* __restrict__ part, int ld_part) {
    pdl_trigger();
    pdl_wait();
    const int n = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (n >= N) return;
    // block storage: logical block (n / 128, k / 64) is 128 x 64 contiguous at its slot
    const int k_blocks = (K + 63) / 64;
    for (int r0 = 0; r0 < rows; r0 += 8) {
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int k0 = lane * 8; k0 < K; k0 += 256) {
            const long long slot = gemm_block_slot((long long)(n >> 7) * k_blocks + (k0 >> 6), total, G);
            const uint4 wv = *(const uint4*)(W + gemm_block_elem(slot, n & 127, k0 & 63));
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

// segment counts of a prompt-pass projection whose last tiles alone are cut along K
__global__ void fill_tail_segs_kernel(int* segs, int m_tiles, int first_cut, int parts) {
    pdl_trigger();
    pdl_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < m_tiles) segs[i] = i >= first_cut ? parts : 1;
}

// rows [from, from + 8) of the normalised activations -> rows [0, 8)
__global__ void move_rows_kernel(bf16* __restrict__ h_hi, bf16* __restrict__ h_lo, int from, int d) {
    pdl_trigger();
    pdl_wait();
    if (from == 0) return;
    const int r = blockIdx.x;
    for (int i = threadIdx.x; i < d / 8; i += blockDim.x) {
        ((uint4*)(h_hi + (size_t)r * d))[i] = ((const uint4*)(h_hi + (size_t)(from + r) * d))[i];
        ((uint4*)(h_lo + (size_t)r * d))[i] = ((const uint4*)(h_lo + (size_t)(from + r) * d))[i];
    }
}

// One projection of the forward.  Returns the per-tile segment counts its consumer must use.
anpd_status gemm_enqueue(anpd_model* m, anpd_kv* kv, int kind, int layer, int rows, const int** seg_count_out, int* seg_max_out = nullptr) {
    int seg_max_dummy;
    if (!seg_max_out) seg_max_out = &seg_max_dummy;
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
        *seg_max_out = 1;
        return gemm_plain_enqueue(plan, W, a_hi, a_lo, rows, ws.part, ws.n_max_out, m->stream, &m->prof);
    }
    if (mode == 1) {                                   // a prompt pass: complete sums, one per output
        const int n_ft = (plan.m_tiles + 1) / 2, n_tt = (rows + 255) / 256;
        const PfSchedule sched = gemm_pf_schedule(n_ft, n_tt, plan.k_blocks, m->num_sms);
        if (sched.tail_split > 1) {                    // feature tiles from `first` on come in tail_split parts, the others in one
            const int first = 2 * (sched.tail_from / n_tt), cfg = first * 4 + sched.tail_split;
            if (m->tail_cfg[kind] != cfg) {
                LAUNCH(&m->prof, m->stream, KC_OTHER, 0,
                       (launch_k(fill_tail_segs_kernel, (plan.m_tiles + 127) / 128, 128, 0, m->stream, m->d_tail_segs[kind], plan.m_tiles, first,
                                 sched.tail_split)));
                m->tail_cfg[kind] = cfg;
            }
            *seg_count_out = m->d_tail_segs[kind];
        } else {
            *seg_count_out = m->d_const_segs[sched.ksplit];
        }
        *seg_max_out = std::max(sched.ksplit, sched.tail_split);
        return gemm_pf_enqueue(plan, W, maps[0], maps[1], rows, ws.part, ws.n_max_out, (size_t)ws.r_max * ws.n_max_out, sched, m->num_sms,
                               ws.gemm_err, m->stream, &m->prof);
    }
    ANPD_TRY(gemm_tc_enqueue(plan, W, maps[0], maps[1], rows, ws.nb[mode], ws.part, (size_t)kv->batch * ANPD_ROWS * ws.n_max_out,
                             ws.n_max_out, ws.gemm_err, m->stream, &m->prof));
    *seg_count_out = plan.d_seg_count;
    *seg_max_out = plan.max_segs;
    return ANPD_OK;
}

template <int HD>
anpd_status attn_enqueue(anpd_model* m, anpd_kv* kv, int layer, int rows, int max_pos, unsigned char* img = nullptr, bool tree = false) {
    const anpd_model_config& c = m->cfg;
    Workspace& ws = kv->ws;
    const size_t layer_elems = (size_t)kv->total_pages * c.n_kv_heads * KV_PAGE * HD;
    const int chunks = max_pos / KV_PAGE + 1;
    const size_t smem = (size_t)KV_PAGE * (HD * 2 + 64) + (size_t)HD * (KV_PAGE * 2 + 64);
    static_assert(4 * 16 * (HD + 4) * sizeof(float) <= (size_t)KV_PAGE * (HD * 2 + 64), "merge buffer must fit in the K staging area");
    static bool attr_set[64] = {false};
    if (first_call_on_device(attr_set)) {
        CUDA_TRY(cudaFuncSetAttribute(attn_partial_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    }
    // a prompt pass: pages are folded in the kernel, nothing to merge (the older 16-row kernel knows one query head per kv head only)
    if (HD == 128 && kv->attn_tc && rows != kv->batch * ANPD_ROWS && kv->attn_pf) return attn_pf_enqueue(m, kv, layer, rows);
    if (HD == 128 && kv->attn_tc && rows != kv->batch * ANPD_ROWS && c.n_q_heads == c.n_kv_heads) return attn_prompt_enqueue(m, kv, layer, rows);
    if (HD == 128 && kv->attn_tc) {
        ANPD_TRY(attn_tc_enqueue(m, kv, layer, rows, max_pos, tree));
    } else {
        dim3 grid(chunks, c.n_kv_heads, rows / ANPD_ROWS);
        LAUNCH(&m->prof, m->stream, KC_ATTN, 0,
               (launch_k(attn_partial_kernel<HD>, grid, ATTN_THREADS, smem, m->stream, ws.q_hi, ws.q_lo, kv->kpool + layer * layer_elems,
                         kv->vpool + layer * layer_elems, kv->page_table, kv->pages_per_seq, ws.row_pos, ws.row_seq, c.n_q_heads,
                         c.n_kv_heads, ws.attn_m, ws.attn_l, ws.attn_o, tree ? ws.row_slot : (const int*)nullptr,
                         tree ? ws.row_hole_lo : (const int*)nullptr, tree ? ws.row_hole_hi : (const int*)nullptr)));
    }
    if (rows >= 64) LAUNCH(&m->prof, m->stream, KC_ATTN, 0,
           (launch_k(attn_combine_wide_kernel<HD / 32>, dim3(rows, c.n_q_heads), 32 * COMBINE_SLICES, 0, m->stream, ws.attn_m, ws.attn_l, ws.attn_o,
                     tree ? ws.row_slot : ws.row_pos, c.n_q_heads, kv->pages_per_seq, ws.ao_hi, ws.ao_lo)));
    else LAUNCH(&m->prof, m->stream, KC_ATTN, 0,
           (launch_k(attn_combine_kernel, dim3(rows, c.n_q_heads), HD * COMBINE_SLICES, 0, m->stream, ws.attn_m, ws.attn_l, ws.attn_o, tree ? ws.row_slot : ws.row_pos, c.n_q_heads,
                                                                              HD, kv->pages_per_seq, ws.ao_hi, ws.ao_lo, img)));
    return ANPD_OK;
}

}  // namespace

anpd_status gemm_plain_enqueue(const GemmPlan& p, const bf16* W, const bf16* a_hi, const bf16* a_lo, int rows, float* part, int ld_part,
                               cudaStream_t st, Profiler* prof) {
    LAUNCH(prof, st, KC_GEMM, 2.0 * (double)p.N * (double)p.K,
           (launch_k(gemm_rows8_kernel, (p.N + 7) / 8, 256, 0, st, W, a_hi, a_lo, rows, p.N, p.K, (long long)p.m_tiles * p.k_blocks, p.grid,
                                                           part, ld_part)));
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}

anpd_status plan_decode_enqueue(anpd_model* m, anpd_kv* kv, bool two_candidates) {
    Workspace& ws = kv->ws;
    LAUNCH(&m->prof, m->stream, KC_OTHER, 0,
           (launch_k(plan_decode_kernel, kv->batch, ANPD_ROWS, 0, m->stream, kv->seq, ws.row_tok, ws.row_pos, ws.row_seq, ws.row_ok,
                                                                      ws.row_slot, ws.row_hole_lo, ws.row_hole_hi, m->cfg.vocab, kv->max_len,
                                                                      two_candidates ? 1 : 0)));
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}

anpd_status plan_prefill_enqueue(anpd_model* m, anpd_kv* kv, int seq, int start, int prompt_len, int rows) {
    Workspace& ws = kv->ws;
    LAUNCH(&m->prof, m->stream, KC_OTHER, 0,
           (launch_k(plan_prefill_kernel, (rows + 127) / 128, 128, 0, m->stream, kv->d_prompt, seq, start, prompt_len, rows, ws.row_tok,
                                                                          ws.row_pos, ws.row_seq, ws.row_ok, ws.row_slot, ws.row_hole_lo,
                                                                          ws.row_hole_hi, m->cfg.vocab, kv->max_len, kv->seq)));
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}

anpd_status accept_enqueue(anpd_model* m, anpd_kv* kv, int mode, const NgramDev* d_ctxs, int seq, int last_row, int prompt_len, bool two_candidates) {
    Workspace& ws = kv->ws;
    const int blocks = (mode == ACCEPT_PREFILL) ? 1 : kv->batch;
    LAUNCH(&m->prof, m->stream, KC_OTHER, 0,
           (launch_k(accept_kernel, blocks, 256, 0, m->stream, kv->seq, ws.amax_val_use, ws.amax_idx_use,
                     ws.amax_nblk, mode, d_ctxs, seq, last_row, prompt_len, two_candidates ? 1 : 0)));
    if (two_candidates && mode == ACCEPT_COMMIT) {
        const anpd_model_config& c = m->cfg;
        LAUNCH(&m->prof, m->stream, KC_OTHER, 0,
               (launch_k(kv_move_kernel, dim3(c.n_layers * c.n_kv_heads, kv->batch), c.head_dim, 0, m->stream, (const SeqState*)kv->seq,
                         (const int*)kv->page_table, kv->pages_per_seq, c.n_kv_heads, c.head_dim,
                         (size_t)kv->total_pages * c.n_kv_heads * KV_PAGE * c.head_dim, kv->kpool, kv->vpool)));
    }
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}

// The forward of a single-sequence step (8 rows) on the row-range projections: per layer QKV (+ rotary, append) ->
// attention -> page combine -> O (+ residual) -> gate/up (+ SwiGLU) -> down (+ residual); then the LM head (+ argmax).
static anpd_status forward_rr_enqueue(anpd_model* m, anpd_kv* kv, int max_pos, bool want_logits) {
    const anpd_model_config& c = m->cfg;
    Workspace& ws = kv->ws;
    cudaStream_t st = m->stream;
    Profiler* pf = &m->prof;
    const int d = c.d_model, hd = c.head_dim;
    const size_t layer_elems = (size_t)kv->total_pages * c.n_kv_heads * KV_PAGE * hd;
    LAUNCH(pf, st, KC_OTHER, 0, (launch_k(embed_img_kernel, ANPD_ROWS, NORM_THREADS, 0, st, m->embed, ws.row_tok, m->layers[0].attn_norm, d, ws.x,
                                          ws.img_h, ws.ss_a)));
    int parts_a = 1;                                   // partial sums of squares behind img_h: 1 after the embedding, then the down projection's CTAs
    for (int l = 0; l < c.n_layers; ++l) {
        const anpd_model::LayerRR& w = m->rr_layers[l];
        RREpiHost q;
        q.ss_in = ws.ss_a; q.n_parts_in = parts_a; q.inv_d_in = 1.0f / (float)d; q.eps = c.rms_eps;
        q.row_pos = ws.row_pos; q.row_seq = ws.row_seq; q.row_ok = ws.row_ok; q.rope_cos = kv->rope_cos; q.rope_sin = kv->rope_sin;
        q.page_table = kv->page_table; q.pages_per_seq = kv->pages_per_seq; q.Hq = c.n_q_heads; q.Hkv = c.n_kv_heads; q.hd = hd;
        q.q_scale = 1.4426950408889634f / sqrtf((float)hd);
        q.q_hi = ws.q_hi; q.q_lo = ws.q_lo; q.kpool_l = kv->kpool + l * layer_elems; q.vpool_l = kv->vpool + l * layer_elems;
        ANPD_TRY(rr_enqueue(RR_QKV, m->rr[GK_QKV], w.wqkv, ws.img_h, q, ws.gemm_err, st, pf));
        if (hd == 128) ANPD_TRY(attn_enqueue<128>(m, kv, l, ANPD_ROWS, max_pos, ws.img_ao));
        else ANPD_TRY(attn_enqueue<64>(m, kv, l, ANPD_ROWS, max_pos, ws.img_ao));
        RREpiHost o;
        o.x = ws.x; o.gain = m->layers[l].ffn_norm; o.ss_out = ws.ss_b; o.d = d; o.act_out = ws.img_h2;
        ANPD_TRY(rr_enqueue(RR_RESID, m->rr[GK_O], w.wo, ws.img_ao, o, ws.gemm_err, st, pf));
        RREpiHost gu;
        gu.ss_in = ws.ss_b; gu.n_parts_in = m->rr[GK_O].G; gu.inv_d_in = 1.0f / (float)d; gu.eps = c.rms_eps; gu.act_out = ws.img_act;
        ANPD_TRY(rr_enqueue(RR_GU, m->rr[GK_GU], w.wgu, ws.img_h2, gu, ws.gemm_err, st, pf));
        RREpiHost dn;
        dn.x = ws.x; dn.gain = (l + 1 < c.n_layers) ? m->layers[l + 1].attn_norm : m->final_norm; dn.ss_out = ws.ss_a; dn.d = d;
        dn.act_out = ws.img_h;
        ANPD_TRY(rr_enqueue(RR_RESID, m->rr[GK_DOWN], w.wd, ws.img_act, dn, ws.gemm_err, st, pf));
        parts_a = m->rr[GK_DOWN].G;
    }
    RREpiHost lm;
    lm.ss_in = ws.ss_a; lm.n_parts_in = parts_a; lm.inv_d_in = 1.0f / (float)d; lm.eps = c.rms_eps;
    lm.logits = want_logits ? ws.logits : nullptr; lm.amax_val = ws.amax_val_rr; lm.amax_idx = ws.amax_idx_rr; lm.V = c.vocab;
    ANPD_TRY(rr_enqueue(RR_LM, m->rr[GK_LM], m->rr_lm, ws.img_h, lm, ws.gemm_err, st, pf));
    ws.amax_nblk = m->rr[GK_LM].G;
    ws.amax_val_use = ws.amax_val_rr;
    ws.amax_idx_use = ws.amax_idx_rr;
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}

anpd_status forward_enqueue(anpd_model* m, anpd_kv* kv, int rows, int max_pos, bool head, bool want_logits, int head_row, bool two_candidates) {
    // the two fused variants know nothing of a second candidate's cache slots and mask
    if (m->rr_ready && kv->batch == 1 && rows == ANPD_ROWS && head && !m->plain_gemm && !two_candidates) return forward_rr_enqueue(m, kv, max_pos, want_logits);
    if (kv->step_ready && rows == kv->batch * ANPD_ROWS && head && !m->prof.on && !two_candidates) return step_kernel_enqueue(m, kv, max_pos, want_logits);
    const anpd_model_config& c = m->cfg;
    kv->ws.amax_nblk = kv->ws.amax_blocks;
    kv->ws.amax_val_use = kv->ws.amax_val;
    kv->ws.amax_idx_use = kv->ws.amax_idx;
    Workspace& ws = kv->ws;
    cudaStream_t st = m->stream;
    Profiler* pf = &m->prof;
    const int d = c.d_model, F = c.d_ffn, hd = c.head_dim, V = c.vocab;
    // between the partial sums of an output: the segments of a decode step, the K parts of a prompt pass
    const size_t sstride = (rows == kv->batch * ANPD_ROWS) ? (size_t)kv->batch * ANPD_ROWS * ws.n_max_out : (size_t)ws.r_max * ws.n_max_out;
    const size_t layer_elems = (size_t)kv->total_pages * c.n_kv_heads * KV_PAGE * hd;
    const int* segs = nullptr;
    int seg_max = 1;                                   // the most partial sums a tile of the last projection has

    LAUNCH(pf, st, KC_OTHER, 0, (launch_k(embed_norm_kernel, rows, NORM_THREADS, 0, st, m->embed, ws.row_tok, m->layers[0].attn_norm, c.rms_eps, d,
                                                                      ws.x, ws.h_hi, ws.h_lo)));
    const bool many_rows = rows >= 64;                 // prefill passes: throughput-shaped launches of the small kernels
    const int rope_hpb = many_rows ? 256 / (hd / 2) : 1;            // heads per block of the rotary kernel
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerW& w = m->layers[l];
        ANPD_TRY(gemm_enqueue(m, kv, GK_QKV, l, rows, &segs, &seg_max));
        if (rows != kv->batch * ANPD_ROWS) {            // a prompt pass
            const dim3 grid((rows + ROPE_TILE_ROWS - 1) / ROPE_TILE_ROWS, c.n_q_heads + 2 * c.n_kv_heads);
            const float qs = 1.4426950408889634f / sqrtf((float)hd);
            if (hd == 128) LAUNCH(pf, st, KC_OTHER, 0,
                   (launch_k(qkv_rope_append_tile_kernel<128>, grid, 256, 0, st, ws.part, segs, sstride, ws.n_max_out, rows, ws.row_pos, ws.row_seq, ws.row_ok,
                             kv->rope_cos, kv->rope_sin, kv->page_table, kv->pages_per_seq, c.n_q_heads, c.n_kv_heads, qs, ws.q_hi, ws.q_lo,
                             kv->kpool + l * layer_elems, kv->vpool + l * layer_elems)));
            else LAUNCH(pf, st, KC_OTHER, 0,
                   (launch_k(qkv_rope_append_tile_kernel<64>, grid, 256, 0, st, ws.part, segs, sstride, ws.n_max_out, rows, ws.row_pos, ws.row_seq, ws.row_ok,
                             kv->rope_cos, kv->rope_sin, kv->page_table, kv->pages_per_seq, c.n_q_heads, c.n_kv_heads, qs, ws.q_hi, ws.q_lo,
                             kv->kpool + l * layer_elems, kv->vpool + l * layer_elems)));
        } else
        LAUNCH(pf, st, KC_OTHER, 0,
               (launch_k(qkv_rope_append_kernel, dim3(rows, (c.n_q_heads + 2 * c.n_kv_heads + rope_hpb - 1) / rope_hpb), rope_hpb * (hd / 2), 0, st, 
                   ws.part, segs, sstride, ws.n_max_out, ws.row_pos, ws.row_slot, ws.row_seq, ws.row_ok, kv->rope_cos, kv->rope_sin,
                   kv->page_table, kv->pages_per_seq, c.n_q_heads, c.n_kv_heads, hd, 1.4426950408889634f / sqrtf((float)hd), ws.q_hi,
                   ws.q_lo, kv->kpool + l * layer_elems, kv->vpool + l * layer_elems, seg_max)));
        if (hd == 128) ANPD_TRY(attn_enqueue<128>(m, kv, l, rows, max_pos, nullptr, two_candidates));
        else ANPD_TRY(attn_enqueue<64>(m, kv, l, rows, max_pos, nullptr, two_candidates));
        ANPD_TRY(gemm_enqueue(m, kv, GK_O, l, rows, &segs, &seg_max));
        LAUNCH(pf, st, KC_OTHER, 0,
               (launch_k(resid_norm_kernel, rows, NORM_THREADS, 0, st, ws.x, ws.part, segs, sstride, ws.n_max_out, w.ffn_norm, c.rms_eps, d,
                                                       ws.h_hi, ws.h_lo, seg_max)));
        ANPD_TRY(gemm_enqueue(m, kv, GK_GU, l, rows, &segs, &seg_max));
        if (many_rows) LAUNCH(pf, st, KC_OTHER, 0,
               (launch_k(swiglu_wide_kernel, dim3((F / 4 + 511) / 512, rows), 256, 0, st, ws.part, segs, sstride, ws.n_max_out, F, ws.act_hi,
                         ws.act_lo)));
        else LAUNCH(pf, st, KC_OTHER, 0,
               (launch_k(swiglu_kernel, dim3((F + 255) / 256, rows), 256, 0, st, ws.part, segs, sstride, ws.n_max_out, F, ws.act_hi,
                                                                          ws.act_lo, seg_max)));
        ANPD_TRY(gemm_enqueue(m, kv, GK_DOWN, l, rows, &segs, &seg_max));
        const float* next_gain = (l + 1 < c.n_layers) ? m->layers[l + 1].attn_norm : m->final_norm;
        LAUNCH(pf, st, KC_OTHER, 0,
               (launch_k(resid_norm_kernel, rows, NORM_THREADS, 0, st, ws.x, ws.part, segs, sstride, ws.n_max_out, next_gain, c.rms_eps, d,
                                                       ws.h_hi, ws.h_lo, seg_max)));
    }
    if (!head) { CUDA_TRY(cudaGetLastError()); return ANPD_OK; }
    int head_rows = rows;
    if (rows != kv->batch * ANPD_ROWS) {
        // A prompt pass needs the LM head for its last token only: the group of 8 rows that holds it moves to rows 0-7 and
        // goes through the decode projection (the other rows of that launch are whatever the buffer holds; rows are independent).
        head_rows = kv->batch * ANPD_ROWS;
        LAUNCH(pf, st, KC_OTHER, 0,
               (launch_k(move_rows_kernel, ANPD_ROWS, 256, 0, st, ws.h_hi, ws.h_lo, (head_row / ANPD_ROWS) * ANPD_ROWS, d)));
    }
    ANPD_TRY(gemm_enqueue(m, kv, GK_LM, 0, head_rows, &segs));
    rows = head_rows;
    LAUNCH(pf, st, KC_OTHER, 0,
           (launch_k(argmax_partial_kernel, dim3(ws.amax_blocks, rows), 256, 0, st, ws.part, segs, (size_t)kv->batch * ANPD_ROWS * ws.n_max_out, ws.n_max_out, V,
                                                                             want_logits ? ws.logits : nullptr, ws.amax_val,
                                                                             ws.amax_idx, ws.amax_blocks)));
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}
