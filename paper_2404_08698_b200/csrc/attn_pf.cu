// Causal attention of a prompt pass (Algorithm 1's LLM(prompt)) for head dimension 128, with the query rows on the
// tensor-memory lanes: a CTA takes 128 consecutive rows of one query head through all the pages (of its kv head) those rows
// may see.
//
//   S  = Q_hi K^T + Q_lo K^T      128 rows x 128 keys of a page, both terms into one accumulator (thread = row)
//   m' = rowmax S if that exceeds m by more than 2^8, else m;  P = 2^(S - m')  (hi + lo terms, to shared memory as the next
//                                           product's M operand)
//   O  = O * 2^(m - m') + P_hi V + P_lo V   in tensor memory; rescaled by the row's own thread, and only when some row of the
//                                           warp moved its reference (multiplying by 1 changes nothing)
//
// A row's scores live in the two threads that share the row (both read all 128 scores of a page and find the same maximum;
// each turns 64 of them into weights), so maxima need no exchange between threads and the sums one per tile.  Roles: one thread requests
// the Q tiles and the K / V^T pages (TMA, a ring of three page buffers filled in the order the products use them: K0, K1, V0,
// K2, V1, ...), one thread issues the products (S of page c+1 before O of page c, so that the tensor core works on the next
// scores while the softmax threads work on these), 256 threads do the softmax, the rescaling and the epilogue.  Two score
// accumulators alternate.  Pages are visited in ascending order and a row's result depends on its own position and inputs
// only.  The queries carry log2(e) / sqrt(hd), as everywhere.  Every wait is bounded and reports through the error flag.
#include "internal.h"
#include "tc_ptx.cuh"

#include <algorithm>
#include <math_constants.h>

typedef __nv_bfloat16 bf16;

namespace {

using namespace tc;

constexpr int FA_HD = 128;
constexpr int FA_ROWS = 128;
constexpr int FA_ATOM = 16384;               // 128 rows x 64 bf16, 128-byte swizzle (one TMA box)
constexpr int FA_OPER = 2 * FA_ATOM;         // a 128 x 128 bf16 operand: two boxes
constexpr int FA_RING = 3;
constexpr int FA_THREADS = 320;              // warp 0: loads, warp 1: products + tensor-memory owner, warps 2-9: softmax (two threads per row)
constexpr int FA_SMEM = (4 + FA_RING) * FA_OPER + 1024;      // Q hi, Q lo, P hi, P lo, three page buffers
constexpr int FA_ERR_TIMEOUT = 206;
constexpr float FA_LAZY = 8.0f;             // base-2 exponent by which a page's maximum must exceed the reference to move it

__device__ __forceinline__ void fa_fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// byte offset of element (row, k) of a 128-row K-major operand made of two 64-column boxes
__device__ __forceinline__ int fa_offset(int row, int k) {
    const int kk = k & 63;
    return (k >> 6) * FA_ATOM + (row >> 3) * 1024 + (row & 7) * 128 + (((kk >> 3) ^ (row & 7)) << 4) + (kk & 7) * 2;
}

struct FaArgs {
    const int* page_table; int pages_per_seq;
    const int* row_pos; const int* row_seq;
    int H, Hkv, layer_row0, rows, n_row_tiles;      // query heads, kv heads (H a multiple of Hkv)
    bf16* ao_hi; bf16* ao_lo;
    int* err;
};

__global__ void __launch_bounds__(FA_THREADS, 1)
attn_pf_kernel(const __grid_constant__ CUtensorMap map_qh, const __grid_constant__ CUtensorMap map_ql,
               const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const FaArgs g) {
    extern __shared__ __align__(1024) unsigned char fa_smem_raw[];
    __shared__ uint64_t q_full, q_empty, ring_full[FA_RING], ring_empty[FA_RING], s_full[2], s_empty[2], p_full, o_done, o_free;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ float l_part[FA_ROWS];

    pdl_trigger();
    unsigned char* smem = fa_smem_raw + ((1024u - (smem_u32(fa_smem_raw) & 1023u)) & 1023u);
    unsigned char* Qh = smem;
    unsigned char* Ql = smem + FA_OPER;
    unsigned char* Ph = smem + 2 * FA_OPER;
    unsigned char* Pl = smem + 3 * FA_OPER;
    unsigned char* ring = smem + 4 * FA_OPER;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(&q_full, 1); mbar_init(&q_empty, 1);
        for (int i = 0; i < FA_RING; ++i) { mbar_init(&ring_full[i], 1); mbar_init(&ring_empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&s_full[i], 1); mbar_init(&s_empty[i], 8); }
        mbar_init(&p_full, 8); mbar_init(&o_done, 1); mbar_init(&o_free, 8);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fa_fence_async_smem();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *((volatile uint32_t*)&tmem_slot);
    const uint32_t tm_s0 = tmem_base, tm_o = tmem_base + 256u;          // S buffers at columns 0 and 128, O at 256
    volatile int* abortp = &abort_flag;

    pdl_wait();                                        // the row plan, the queries and this pass's K/V rows come from earlier kernels

    // work items: (row tile, head), the tiles with the most pages first
    // The CTAs take the items round by round, every other round in reverse CTA order, so that the CTA with the longest item
    // of one round gets the shortest of the next.
    const int n_items = g.n_row_tiles * g.H;
    auto nth = [&](int k) -> int {                       // this CTA's k-th item (>= n_items: none)
        const int G = (int)gridDim.x;
        return k * G + ((k & 1) ? G - 1 - (int)blockIdx.x : (int)blockIdx.x);
    };
    auto item = [&](int it, int& r0, int& h, int& n_pages, int& seq, int& pos_lo) {
        const int rt = g.n_row_tiles - 1 - it / g.H;
        h = it % g.H;
        r0 = rt * FA_ROWS;
        const int last = min(r0 + FA_ROWS, g.rows) - 1;
        pos_lo = g.row_pos[r0];
        n_pages = g.row_pos[last] / KV_PAGE + 1;
        seq = g.row_seq[r0];
    };

    if (warp == 0) {
        // ---------------- loads ----------------
        if (lane == 0) {
            const uint64_t pol = policy_evict_last();               // a page is read by every row tile behind it
            uint32_t tq = 0, li = 0;                                // tiles begun, page loads issued so far
            bool ok = true;
            for (int k = 0, it = nth(0); it < n_items && ok; ++k, it = nth(k), ++tq) {
                int r0, h, n_pages, seq, pos_lo;
                item(it, r0, h, n_pages, seq, pos_lo);
                ok = mbar_wait(&q_empty, (tq & 1u) ^ 1u, abortp);
                if (!ok) break;
                mbar_expect_tx(&q_full, 2 * FA_OPER);
                tma_load_2d(Qh, &map_qh, h * FA_HD, r0, &q_full, pol);
                tma_load_2d(Qh + FA_ATOM, &map_qh, h * FA_HD + 64, r0, &q_full, pol);
                tma_load_2d(Ql, &map_ql, h * FA_HD, r0, &q_full, pol);
                tma_load_2d(Ql + FA_ATOM, &map_ql, h * FA_HD + 64, r0, &q_full, pol);
                // K0, then for every page c: K(c+1) if there is one, V(c)
                for (int j = 0; j < 2 * n_pages && ok; ++j, ++li) {
                    // j = 0: K0; odd j: K((j+1)/2) while it exists; even j > 0: V(j/2 - 1); the tail: V(n-1)
                    int c;
                    bool kk;
                    if (j == 0) { kk = true; c = 0; }
                    else if (j == 2 * n_pages - 1) { kk = false; c = n_pages - 1; }
                    else if (j & 1) { kk = true; c = (j + 1) / 2; }
                    else { kk = false; c = j / 2 - 1; }
                    const uint32_t slot = li % FA_RING, use = li / FA_RING;
                    ok = mbar_wait(&ring_empty[slot], (use & 1u) ^ 1u, abortp);
                    if (!ok) break;
                    const int row = g.layer_row0 + (g.page_table[seq * g.pages_per_seq + c] * g.Hkv + h / (g.H / g.Hkv)) * KV_PAGE;
                    unsigned char* dst = ring + (size_t)slot * FA_OPER;
                    mbar_expect_tx(&ring_full[slot], FA_OPER);
                    tma_load_2d(dst, kk ? &map_k : &map_v, 0, row, &ring_full[slot], pol);
                    tma_load_2d(dst + FA_ATOM, kk ? &map_k : &map_v, 64, row, &ring_full[slot], pol);
                }
            }
            if (!ok) {
                // gave up: let the copies already requested land before the CTA may exit
                for (uint32_t b = 0; b < FA_RING && b < li; ++b) {
                    const uint32_t idx = li - 1 - b;
                    for (unsigned spin = 0; spin < WAIT_LIMIT && !mbar_try_wait(&ring_full[idx % FA_RING], (idx / FA_RING) & 1u); ++spin) {}
                }
                if (tq) for (unsigned spin = 0; spin < WAIT_LIMIT && !mbar_try_wait(&q_full, (tq - 1) & 1u); ++spin) {}
            }
        }
    } else if (warp == 1) {
        // ---------------- products ----------------
        if (lane == 0) {
            // fp32 accumulate, bf16 x bf16, both operands K-major, M = 128, N = 128
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
            uint32_t tq = 0, li = 0, pc = 0;                        // tiles, page loads consumed, pages whose S was issued
            uint32_t pv = 0;                                        // pages whose O product was issued
            bool ok = true;
            auto product = [&](uint32_t d_tmem, const unsigned char* a_hi, const unsigned char* a_lo, const unsigned char* b, uint32_t acc) {
                // D (+)= A_hi B^T + A_lo B^T over the 128-wide contraction: 8 steps of 16 per term
#pragma unroll
                for (int term = 0; term < 2; ++term) {
                    const unsigned char* a = term ? a_lo : a_hi;
#pragma unroll
                    for (int k16 = 0; k16 < 8; ++k16) {
                        const uint64_t adv = (uint64_t)((k16 & 3) * 2);
                        tc_mma_bf16(d_tmem, make_smem_desc(smem_u32(a + (k16 >> 2) * FA_ATOM)) + adv,
                                    make_smem_desc(smem_u32(b + (k16 >> 2) * FA_ATOM)) + adv, idesc, (acc | term | k16) ? 1u : 0u);
                    }
                }
            };
            for (int k = 0, it = nth(0); it < n_items && ok; ++k, it = nth(k), ++tq) {
                int r0, h, n_pages, seq, pos_lo;
                item(it, r0, h, n_pages, seq, pos_lo);
                ok = mbar_wait(&q_full, tq & 1u, abortp);
                if (!ok) break;
                auto scores = [&]() -> bool {                       // S of the next page in line
                    const uint32_t slot = li % FA_RING, use = li / FA_RING, b = pc & 1u;
                    if (!mbar_wait(&ring_full[slot], use & 1u, abortp)) return false;
                    if (!mbar_wait(&s_empty[b], ((pc >> 1) & 1u) ^ 1u, abortp)) return false;
                    tc_fence_after();
                    product(tm_s0 + b * 128u, Qh, Ql, ring + (size_t)slot * FA_OPER, 0u);
                    tc_commit(&ring_empty[slot]);
                    tc_commit(&s_full[b]);
                    ++li; ++pc;
                    return true;
                };
                ok = scores();
                for (int c = 0; c < n_pages && ok; ++c) {
                    if (c + 1 < n_pages) { ok = scores(); if (!ok) break; }
                    const uint32_t slot = li % FA_RING, use = li / FA_RING;
                    ok = mbar_wait(&ring_full[slot], use & 1u, abortp);
                    if (!ok) break;
                    if (c == 0) { ok = mbar_wait(&o_free, (tq & 1u) ^ 1u, abortp); if (!ok) break; }      // the last tile's output has been read
                    ok = mbar_wait(&p_full, pv & 1u, abortp);
                    if (!ok) break;
                    tc_fence_after();
                    product(tm_o, Ph, Pl, ring + (size_t)slot * FA_OPER, c > 0 ? 1u : 0u);
                    tc_commit(&ring_empty[slot]);
                    tc_commit(&o_done);
                    ++li; ++pv;
                }
                if (ok) tc_commit(&q_empty);                        // every product that reads this tile's Q has been issued
            }
        }
    } else {
        // ---------------- softmax, rescaling, epilogue: two threads per row ----------------
        // Both threads of a row read all its 128 scores and find the same maximum; each then turns its own 64 keys into
        // weights, rescales and finally writes its own 64 output dimensions; the two halves of the weights' sum meet once
        // per tile.
        const int quad = warp & 3;                        // a warp may only touch tensor-memory lanes 32 * (warp % 4) .. + 31
        const int half = (warp - 2) >> 2;                 // warps 2-5: keys / dimensions 0-63, warps 6-9: 64-127
        const int r = quad * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        uint32_t pc = 0, od = 0;                          // pages begun, completions of the O product consumed
        bool ok = true;
        for (int k = 0, it = nth(0); it < n_items && ok; ++k, it = nth(k)) {
            int r0, h, n_pages, seq, pos_lo;
            item(it, r0, h, n_pages, seq, pos_lo);
            const int row = r0 + r;
            const int pos = row < g.rows ? g.row_pos[row] : -1;         // -1: a padding row sees no key
            float m_run = -CUDART_INF_F, l_run = 0.0f;
            for (int c = 0; c < n_pages && ok; ++c, ++pc) {
                const uint32_t b = pc & 1u;
                ok = mbar_wait(&s_full[b], (pc >> 1) & 1u, abortp);
                if (!ok) break;
                tc_fence_after();
                const uint32_t ts = tm_s0 + b * 128u + lane_addr;
                const int key0 = c * KV_PAGE;
                const bool any_masked = __any_sync(0xffffffffu, key0 + KV_PAGE - 1 > pos);     // some key of the page is hidden from a row of this warp
                // the row's maximum over the page (all 128 scores), and this thread's 64 scores
                float sv[64];
                float mx;
                {
                    float all[KV_PAGE];
                    tc_ld128(ts, all);
                    if (any_masked) {
#pragma unroll
                        for (int i = 0; i < KV_PAGE; ++i) all[i] = (key0 + i > pos) ? -CUDART_INF_F : all[i];
                    }
                    float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
                    for (int i = 0; i < KV_PAGE; ++i) mx4[i & 3] = fmaxf(mx4[i & 3], all[i]);
                    mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
#pragma unroll
                    for (int i = 0; i < 64; ++i) sv[i] = half ? all[64 + i] : all[i];
                }
                // The reference maximum follows the row's maximum lazily: it moves only when the page's maximum exceeds it by
                // more than 2^8 (the weights are 2^(S - m'), so they stay below 2^8: exact in fp32 and in the hi + lo terms;
                // the final division by the weights' sum removes the reference).  Most pages then need no rescaling of O.
                const bool raise = mx > m_run + FA_LAZY;            // also true while m_run is -inf and the row sees a key
                const float m_new = raise ? mx : m_run;
                const float scale = !raise ? 1.0f : (m_run == -CUDART_INF_F ? 0.0f : exp2f(m_run - m_new));
                // the P operand and O are free once the previous page's second product is done
                if (c > 0) {
                    ok = mbar_wait(&o_done, od & 1u, abortp);
                    ++od;
                    if (!ok) break;
                    tc_fence_after();
                    if (__any_sync(0xffffffffu, scale != 1.0f)) {
#pragma unroll 1
                        for (int ch = 0; ch < 2; ++ch) {
                            float o[32];
                            tc_ld32(tm_o + lane_addr + (uint32_t)(half * 64 + ch * 32), o);
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] *= scale;
                            tc_st32(tm_o + lane_addr + (uint32_t)(half * 64 + ch * 32), o);
                        }
                    }
                }
                // weights: P = 2^(S - m') as hi + lo terms; 2^(-inf) is 0, and a row that has seen no key yet has only -inf scores
                const float m_use = (m_new == -CUDART_INF_F) ? 0.0f : m_new;
                float sum = 0.0f;
#pragma unroll
                for (int i0 = 0; i0 < 64; i0 += 8) {
                    __nv_bfloat162 hh[4], ll[4];
#pragma unroll
                    for (int i = 0; i < 8; i += 2) {
                        float p0, p1;
                        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(p0) : "f"(sv[i0 + i] - m_use));
                        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(p1) : "f"(sv[i0 + i + 1] - m_use));
                        sum += p0;
                        sum += p1;
                        hh[i >> 1] = __floats2bfloat162_rn(p0, p1);
                        const float2 back = __bfloat1622float2(hh[i >> 1]);
                        ll[i >> 1] = __floats2bfloat162_rn(p0 - back.x, p1 - back.y);
                    }
                    const int off = fa_offset(r, half * 64 + i0);
                    *(uint4*)(Ph + off) = *(const uint4*)hh;
                    *(uint4*)(Pl + off) = *(const uint4*)ll;
                }
                l_run = fmaf(l_run, scale, sum);
                m_run = m_new;
                fa_fence_async_smem();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&p_full); mbar_arrive(&s_empty[b]); }
            }
            if (!ok) break;
            // the two halves of the weights' sum (always added in the same order)
            if (half == 1) l_part[r] = l_run;
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (half == 0) l_part[r] = l_run + l_part[r];
            asm volatile("bar.sync 1, 256;" ::: "memory");
            const float l_tot = l_part[r];
            // the tile's last product, then O / l as hi + lo terms straight to the O projection's input
            ok = mbar_wait(&o_done, od & 1u, abortp);
            ++od;
            if (!ok) break;
            tc_fence_after();
#pragma unroll 1
            for (int ch = 0; ch < 2; ++ch) {
                float o[32];
                tc_ld32(tm_o + lane_addr + (uint32_t)(half * 64 + ch * 32), o);
                if (row < g.rows) {
                    __nv_bfloat162 hh[16], ll[16];
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        const float t0 = o[i] / l_tot, t1 = o[i + 1] / l_tot;
                        hh[i >> 1] = __floats2bfloat162_rn(t0, t1);
                        const float2 back = __bfloat1622float2(hh[i >> 1]);
                        ll[i >> 1] = __floats2bfloat162_rn(t0 - back.x, t1 - back.y);
                    }
                    const size_t out = (size_t)row * g.H * FA_HD + (size_t)h * FA_HD + half * 64 + ch * 32;
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        *(uint4*)(g.ao_hi + out + 8 * u) = *(const uint4*)(hh + 4 * u);
                        *(uint4*)(g.ao_lo + out + 8 * u) = *(const uint4*)(ll + 4 * u);
                    }
                }
            }
            tc_fence_before();
            asm volatile("bar.sync 1, 256;" ::: "memory");       // both halves have read l_part and O before either is written again
            if (lane == 0) mbar_arrive(&o_free);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
    if (threadIdx.x == 0 && abort_flag) atomicExch(g.err, FA_ERR_TIMEOUT);
}

}  // namespace

// Attention of a prompt pass over `rows` rows (a multiple of 8; the row plan covers the padding) of sequence row_seq[0].
// map_qh / map_ql: the pass's queries [rows][H * 128] seen through boxes of 64 columns x 128 rows.
anpd_status attn_pf_enqueue(anpd_model* m, anpd_kv* kv, int layer, int rows) {
    const anpd_model_config& c = m->cfg;
    Workspace& ws = kv->ws;
    static bool attr_set[64] = {false};
    if (first_call_on_device(attr_set)) {
        CUDA_TRY(cudaFuncSetAttribute(attn_pf_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FA_SMEM));
    }
    FaArgs g;
    g.page_table = kv->page_table; g.pages_per_seq = kv->pages_per_seq;
    g.row_pos = ws.row_pos; g.row_seq = ws.row_seq;
    g.H = c.n_q_heads; g.Hkv = c.n_kv_heads;
    g.layer_row0 = layer * kv->total_pages * c.n_kv_heads * KV_PAGE;
    g.rows = rows;
    g.n_row_tiles = (rows + FA_ROWS - 1) / FA_ROWS;
    g.ao_hi = ws.ao_hi; g.ao_lo = ws.ao_lo;
    g.err = ws.gemm_err;
    const int grid = std::min(m->num_sms, g.n_row_tiles * g.H);
    LAUNCH(&m->prof, m->stream, KC_ATTN, 0,
           (launch_k(attn_pf_kernel, grid, FA_THREADS, (size_t)FA_SMEM, m->stream, ws.map_q[0], ws.map_q[1], kv->map_k, kv->map_v, g)));
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}
