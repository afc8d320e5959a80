// Attention of the verify step for head dimension 128 on the sm_100a tensor cores
// (paper Section 3.1, "Verification": the K+1 rows of a step attend to the cached keys).
//
// A work item is one 128-key page of one kv head for one group of 8 rows.  With so few query rows
// the operands are swapped, as in the weight GEMM: the page is the MMA's 128-row M operand and the
// 8 x G query vectors that share the kv head are its N operand.
//   S^T [128 keys x N]  = K page   [128 keys x 128 dims] . Q^T     (tcgen05.mma, accumulator in tensor memory)
//   O^T [128 dims x N]  = V^T page [128 dims x 128 keys] . P^T
// K pages are stored [key][dim] and V pages transposed [dim][key], so both are K-major and arrive by
// TMA in the 128-byte-swizzled layout the MMA reads.  Queries and softmax weights enter as two bf16
// terms each (hi rows then lo rows of the N operand, N = 2 x 8 x G), so only the cache's own bf16
// rounding is left; the two halves of an accumulator are added when it is read back.
//
// The kernel is persistent: one CTA per SM holds up to five independent "slots" (a warpgroup of
// 128 threads with its own 32 KB page buffer, operand staging and tensor-memory columns), and a
// slot walks through its share of the items.  The page buffer first receives the K page; as soon as
// the first product has consumed it the V^T page is requested into the same buffer and lands while
// the softmax runs; after the second product the next item's K page follows.  With four or five slots
// per SM every SM keeps several page copies in flight, and at the context lengths of interest each slot
// has one or two items.
// Thread t of a slot owns tensor-memory lane t: key t of the page after the first product, output
// dimension t after the second.  The softmax over the page's keys is a reduction across threads
// (shuffle tree inside a warp, then the four warps in warp order).  Each page leaves a partial
// (max, sum, weighted values) per query vector; the combine kernel merges pages in page order.
// Every value depends on the row's own position and inputs only: masked keys contribute exact zeros
// and the order of every sum is fixed by key positions, so a row's result does not depend on which
// other rows share the launch, nor on which slot handled the page.
#include "internal.h"
#include "tc_ptx.cuh"

#include <math_constants.h>

#include <algorithm>
#include <cstdlib>

typedef __nv_bfloat16 bf16;

namespace {

using namespace tc;

constexpr int HD = 128;
constexpr int PAGE_ATOM = 128 * 128;        // bytes of a 128-row x 64-column bf16 tile (one TMA box)
constexpr int ATTN_ERR_TIMEOUT = 202;

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Byte offset of element (row n, column k) of an [N rows][128 columns] bf16 operand held as two
// 64-column tiles in the 128-byte-swizzled K-major layout (8-row groups 1024 bytes apart).
template <int N>
__device__ __forceinline__ int b_operand_offset(int n, int k) {
    const int kk = k & 63;
    return (k >> 6) * (N * 128) + (n >> 3) * 1024 + (n & 7) * 128 + ((((kk >> 3) ^ (n & 7))) << 4) + (kk & 7) * 2;
}

// S slots per CTA for G query heads per kv head (bounded by shared memory and tensor memory).
template <int G, int S> struct AttnCfg {
    static constexpr int Q = 8 * G;                      // query vectors: 8 rows x G heads of the group
    static constexpr int N = 2 * Q;                      // MMA N: hi terms then lo terms
    static constexpr int B_BYTES = N * 256;              // one N-row operand (two 64-column tiles)
    static constexpr int SLOT_BYTES = 2 * PAGE_ATOM + 2 * B_BYTES;       // page buffer (K, then V), Q operand, P operand
    static constexpr int SLOTS = S;
    static constexpr int THREADS = SLOTS * 128;
    static constexpr int TMEM_NEED = SLOTS * N;          // per slot N columns: S^T, then O^T in the same columns
    static constexpr int TMEM_COLS = TMEM_NEED <= 32 ? 32 : TMEM_NEED <= 64 ? 64 : TMEM_NEED <= 128 ? 128 : TMEM_NEED <= 256 ? 256 : 512;
    static constexpr size_t SMEM = (size_t)SLOTS * SLOT_BYTES + 1024;
};

__device__ __forceinline__ void slot_bar(int slot) { asm volatile("bar.sync %0, 128;" ::"r"(slot + 1) : "memory"); }

struct AttnItem { int c, kvh, r0, pos_lo, seq; };

template <int G, int S>
__global__ void __launch_bounds__(AttnCfg<G, S>::THREADS, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const bf16* __restrict__ q_hi,
               const bf16* __restrict__ q_lo, const int* __restrict__ page_table, int pages_per_seq, const int* __restrict__ row_pos,
               const int* __restrict__ row_seq, int Hq, int Hkv, int layer_row0, int chunks, int n_items, float* __restrict__ pm,
               float* __restrict__ pl, float* __restrict__ po, int* err, const int* __restrict__ row_slot,
               const int* __restrict__ row_hole_lo, const int* __restrict__ row_hole_hi) {
    // row_slot / row_hole_*: null except in two-candidate steps, where row r of a group lives in cache slot pos_lo + r, its
    // group reaches up to row_slot[last row], and a second candidate's rows must not see the slots [hole_lo, hole_hi)
    typedef AttnCfg<G, S> Cfg;
    constexpr int Q = Cfg::Q, N = Cfg::N, SLOTS = Cfg::SLOTS;
    extern __shared__ __align__(1024) unsigned char attn_tc_smem[];
    __shared__ uint64_t bar_k[SLOTS], bar_v[SLOTS], bar_s[SLOTS], bar_o[SLOTS];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ float red_max[SLOTS][4][Q];
    __shared__ float red_sum[SLOTS][2][4][Q];

    pdl_trigger();
    const int slot = threadIdx.x >> 7, t = threadIdx.x & 127, warp = t >> 5, lane = t & 31;
    unsigned char* smem = attn_tc_smem + ((1024u - (smem_u32(attn_tc_smem) & 1023u)) & 1023u) + (size_t)slot * Cfg::SLOT_BYTES;
    unsigned char* Bs = smem;                        // the K page (tiles: dims 0..63, 64..127), later the V^T page (keys 0..63, 64..127)
    unsigned char* Qs = smem + 2 * PAGE_ATOM;
    unsigned char* Ps = Qs + Cfg::B_BYTES;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int i = 0; i < SLOTS; ++i) { mbar_init(&bar_k[i], 1); mbar_init(&bar_v[i], 1); mbar_init(&bar_s[i], 1); mbar_init(&bar_o[i], 1); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"((uint32_t)Cfg::TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *((volatile uint32_t*)&tmem_slot) + (uint32_t)(slot * N);
    const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
    volatile int* abortp = &abort_flag;
    // fp32 accumulate, bf16 x bf16, both operands K-major, M = 128
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
    const uint64_t pol = policy_evict_first();

    pdl_wait();                                      // the row plan, the queries and this step's K/V rows come from earlier kernels

    // Item `it` -> (page, kv head, row group); pages beyond the group's last position hold nothing a row may see.
    const int stride = gridDim.x * SLOTS;
    auto decode = [&](int it, AttnItem& out) {
        const int rest = it / chunks;
        out.c = it % chunks; out.kvh = rest % Hkv; out.r0 = (rest / Hkv) * ANPD_ROWS;
    };
    auto next_item = [&](int it, AttnItem& out) -> int {
        for (; it < n_items; it += stride) {
            decode(it, out);
            const int hi = (row_slot ? row_slot : row_pos)[out.r0 + ANPD_ROWS - 1];          // three independent loads
            out.pos_lo = row_pos[out.r0];
            out.seq = row_seq[out.r0];
            if (out.c * KV_PAGE <= hi) return it;
        }
        return n_items;
    };
    auto page_row = [&](const AttnItem& a) -> int {   // first row of the item's page in the pools' 2-D view
        return layer_row0 + (page_table[a.seq * pages_per_seq + a.c] * Hkv + a.kvh) * KV_PAGE;
    };
    auto load_page = [&](const CUtensorMap* map, uint64_t* bar, const AttnItem& a) {
        const int row = page_row(a);
        mbar_expect_tx(bar, 2 * PAGE_ATOM);
        tma_load_2d(Bs, map, 0, row, bar, pol);
        tma_load_2d(Bs + PAGE_ATOM, map, 64, row, bar, pol);
    };
    // queries: row n of the operand is query vector n % Q (hi term for n < Q, lo term after); 16-byte chunks
    constexpr int QCH = (N * 16 + 127) / 128;
    auto fetch_q = [&](const AttnItem& a, uint4* regs) {
#pragma unroll
        for (int u = 0; u < QCH; ++u) {
            const int idx = t + u * 128;
            if (idx < N * 16) {
                const int n = idx >> 4, c16 = idx & 15;
                const int qn = n % Q, g = qn >> 3, r = qn & 7;
                const bf16* src = (n < Q ? q_hi : q_lo) + (size_t)(a.r0 + r) * Hq * HD + (size_t)(a.kvh * G + g) * HD + c16 * 8;
                regs[u] = *(const uint4*)src;
            }
        }
    };
    auto stage_q = [&](const uint4* regs) {
#pragma unroll
        for (int u = 0; u < QCH; ++u) {
            const int idx = t + u * 128;
            if (idx < N * 16) *(uint4*)(Qs + b_operand_offset<N>(idx >> 4, (idx & 15) * 8)) = regs[u];
        }
    };

    AttnItem cur, nxt;
    int it = slot * gridDim.x + blockIdx.x;          // consecutive items go to different SMs: every SM gets its share of slots in use
    uint32_t k_issued = 0, v_issued = 0;             // page loads requested by this slot's first thread
    if (it < n_items) {
        // the queries of the slot's first candidate are requested before anything that has to wait for the row plan
        uint4 qr[QCH];
        decode(it, cur);
        fetch_q(cur, qr);
        const int first = it;
        it = next_item(it, cur);
        if (it < n_items) {
            if (t == 0) { load_page(&map_k, &bar_k[slot], cur); k_issued = 1; }
            if (it != first) fetch_q(cur, qr);
            stage_q(qr);
            fence_async_smem();
            slot_bar(slot);
        }
    }
    for (uint32_t j = 0; it < n_items; ++j) {
        const uint32_t par = j & 1u;
        const int it_next = next_item(it + stride, nxt);
        const bool more = it_next < n_items;
        // ---- S^T = K . Q^T ----
        if (t == 0) {
            if (mbar_wait(&bar_k[slot], par, abortp)) {
                tc_fence_after();
#pragma unroll
                for (int k16 = 0; k16 < HD / 16; ++k16) {
                    const uint64_t adv = (uint64_t)((k16 & 3) * 2);                 // 32 bytes along K inside the swizzle row, 16-byte units
                    tc_mma_bf16(tmem_base, make_smem_desc(smem_u32(Bs + (k16 >> 2) * PAGE_ATOM)) + adv,
                                make_smem_desc(smem_u32(Qs + (k16 >> 2) * (N * 128))) + adv, idesc, k16 > 0 ? 1u : 0u);
                }
                tc_commit(&bar_s[slot]);
            }
        }
        mbar_wait(&bar_s[slot], par, abortp);
        tc_fence_after();
        // the first product is done with the page buffer and the query staging: the V^T page takes the buffer,
        // and the next item's queries are requested
        if (t == 0) { load_page(&map_v, &bar_v[slot], cur); ++v_issued; }
        uint4 qr[QCH];
        if (more) fetch_q(nxt, qr);
        // Scores of this thread's key (c * 128 + t) for QC query vectors at a time, masked by position.  With up to 16
        // query vectors (1 or 2 query heads per kv head) they stay in registers across the barrier; with more they are
        // read from tensor memory a second time instead (the second product overwrites them only after the barrier
        // behind the P operand), which keeps the kernel out of local memory.
        constexpr int QC = Q < 16 ? Q : 16;
        const int key = cur.c * KV_PAGE + t;
        auto scores = [&](int q0, float* s) {
            float v[2 * QC];
            if constexpr (Q <= 8) {
                tc_ld16(lane_base, v);                                           // hi terms 0..7, lo terms 8..15
            } else {
                tc_ld16(lane_base + (uint32_t)q0, v);
                tc_ld16(lane_base + (uint32_t)(Q + q0), v + QC);
            }
#pragma unroll
            for (int q = 0; q < QC; ++q) {
                s[q] = v[q] + v[QC + q];
                if (key > cur.pos_lo + (q & 7)) s[q] = -CUDART_INF_F;           // q0 is a multiple of 8: (q0 + q) & 7 == q & 7
                if (row_slot && key >= row_hole_lo[cur.r0 + (q & 7)] && key < row_hole_hi[cur.r0 + (q & 7)]) s[q] = -CUDART_INF_F;
            }
        };
        float s_keep[QC];
        // maximum over the page's keys per query vector
#pragma unroll
        for (int q0 = 0; q0 < Q; q0 += QC) {
            float s[QC];
            scores(q0, s);
#pragma unroll
            for (int q = 0; q < QC; ++q) {
                float mx = s[q];
                for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                if (lane == 0) red_max[slot][warp][q0 + q] = mx;
                if (Q <= 16) s_keep[q] = s[q];
            }
        }
        tc_fence_before();
        slot_bar(slot);
        if constexpr (Q > 16) tc_fence_after();
        // weights (base-2 domain: the queries carry log2(e) / sqrt(hd)), their sum, and the P operand
#pragma unroll
        for (int q0 = 0; q0 < Q; q0 += QC) {
            float s[QC];
            if constexpr (Q <= 16) {
#pragma unroll
                for (int q = 0; q < QC; ++q) s[q] = s_keep[q];
            } else {
                scores(q0, s);
            }
#pragma unroll
            for (int q = 0; q < QC; ++q) {
                const int qq = q0 + q;
                const float m = fmaxf(fmaxf(red_max[slot][0][qq], red_max[slot][1][qq]), fmaxf(red_max[slot][2][qq], red_max[slot][3][qq]));
                const float p = (m == -CUDART_INF_F) ? 0.0f : exp2f(s[q] - m);
                const bf16 h = __float2bfloat16_rn(p);
                const bf16 l = __float2bfloat16_rn(p - __bfloat162float(h));
                *(bf16*)(Ps + b_operand_offset<N>(qq, t)) = h;
                *(bf16*)(Ps + b_operand_offset<N>(Q + qq, t)) = l;
                float sum = p;
                for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
                if (lane == 0) red_sum[slot][par][warp][qq] = sum;
            }
        }
        if constexpr (Q > 16) tc_fence_before();          // the scores were read again: order those reads before the second product
        if (more) stage_q(qr);
        fence_async_smem();
        slot_bar(slot);
        // ---- O^T = V^T . P^T (into the columns S^T occupied: every thread has read its scores) ----
        if (t == 0) {
            if (mbar_wait(&bar_v[slot], par, abortp)) {
                tc_fence_after();
#pragma unroll
                for (int k16 = 0; k16 < KV_PAGE / 16; ++k16) {
                    const uint64_t adv = (uint64_t)((k16 & 3) * 2);
                    tc_mma_bf16(tmem_base, make_smem_desc(smem_u32(Bs + (k16 >> 2) * PAGE_ATOM)) + adv,
                                make_smem_desc(smem_u32(Ps + (k16 >> 2) * (N * 128))) + adv, idesc, k16 > 0 ? 1u : 0u);
                }
                tc_commit(&bar_o[slot]);
            }
        }
        if (t < Q) {
            const size_t out = ((size_t)(cur.r0 + (t & 7)) * Hq + (cur.kvh * G + (t >> 3))) * pages_per_seq + cur.c;
            pm[out] = fmaxf(fmaxf(red_max[slot][0][t], red_max[slot][1][t]), fmaxf(red_max[slot][2][t], red_max[slot][3][t]));
            pl[out] = (red_sum[slot][par][0][t] + red_sum[slot][par][1][t]) + (red_sum[slot][par][2][t] + red_sum[slot][par][3][t]);
        }
        mbar_wait(&bar_o[slot], par, abortp);
        tc_fence_after();
        if (more && t == 0) { load_page(&map_k, &bar_k[slot], nxt); ++k_issued; }        // the second product is done with the page buffer
#pragma unroll
        for (int q0 = 0; q0 < Q; q0 += QC) {
            float v[2 * QC];
            if constexpr (Q <= 8) {
                tc_ld16(lane_base, v);
            } else {
                tc_ld16(lane_base + (uint32_t)q0, v);
                tc_ld16(lane_base + (uint32_t)(Q + q0), v + QC);
            }
#pragma unroll
            for (int q = 0; q < QC; ++q) {
                const int qq = q0 + q;
                const size_t out = ((size_t)(cur.r0 + (qq & 7)) * Hq + (cur.kvh * G + (qq >> 3))) * pages_per_seq + cur.c;
                po[out * HD + t] = v[q] + v[QC + q];
            }
        }
        tc_fence_before();
        if (more) slot_bar(slot);                    // the next first product overwrites the columns just read
        cur = nxt;
        it = it_next;
    }
    if (t == 0 && abort_flag) {
        // gave up somewhere: let the last page copies land before the CTA may exit
        if (k_issued) for (unsigned spin = 0; spin < WAIT_LIMIT && !mbar_try_wait(&bar_k[slot], (k_issued - 1) & 1u); ++spin) {}
        if (v_issued) for (unsigned spin = 0; spin < WAIT_LIMIT && !mbar_try_wait(&bar_v[slot], (v_issued - 1) & 1u); ++spin) {}
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicExch(err, ATTN_ERR_TIMEOUT);
    if (threadIdx.x < 32) {
        tc_fence_after();
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(*((volatile uint32_t*)&tmem_slot)), "r"((uint32_t)Cfg::TMEM_COLS) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------
// Prompt passes (one query head per kv head): causal attention of a tile of 16 consecutive rows of one head over all the
// pages those rows may see, page after page with a running maximum, so that no per-page partial leaves the SM and no merge
// kernel follows.  Products, operand layouts and the page buffer's K -> V^T -> next K rotation are those of the kernel
// above.  Per page: S^T = K . Q^T; the page's maxima (folded by eight threads per row, through shared memory) raise the
// running maxima m, kept by one thread per row; P = 2^(S - m) (hi + lo) goes to shared
// memory; thread t keeps the sum of its own key's weights, rescaled by 2^(m_old - m) like the output accumulator
// O[q] (thread = output dimension, in registers), to which O^T = V^T . P^T of the page is added.  The weights' sums are
// reduced across threads once, at the end.  Pages are visited in ascending order: the result depends on the row's own
// position and inputs only.
// ---------------------------------------------------------------------------------------------
constexpr int PFQ = 16, PFN = 32;            // rows per tile; MMA N (hi + lo terms)
constexpr int PF_SLOTS = 4;
constexpr int PF_B_BYTES = PFN * 256;
constexpr int PF_SLOT_BYTES = 2 * PAGE_ATOM + 2 * PF_B_BYTES;
constexpr size_t PF_SMEM = (size_t)PF_SLOTS * PF_SLOT_BYTES + 1024;

__global__ void __launch_bounds__(PF_SLOTS * 128, 1)
attn_prompt_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const bf16* __restrict__ q_hi,
                   const bf16* __restrict__ q_lo, const int* __restrict__ page_table, int pages_per_seq, const int* __restrict__ row_pos,
                   const int* __restrict__ row_seq, int H, int layer_row0, int n_tiles, bf16* __restrict__ ao_hi, bf16* __restrict__ ao_lo,
                   int* err) {
    extern __shared__ __align__(1024) unsigned char attn_tc_smem[];
    __shared__ uint64_t bar_k[PF_SLOTS], bar_v[PF_SLOTS], bar_s[PF_SLOTS], bar_o[PF_SLOTS];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ float2 row_ms[PF_SLOTS][PFQ];             // per row: the maximum so far, the factor that rescales older sums to it
    __shared__ float red_sum[PF_SLOTS][4][PFQ];
    static_assert(PFQ * KV_PAGE * sizeof(float) <= PF_B_BYTES && PFQ * 8 == 128, "the scores of a page pass through the P operand's buffer");

    pdl_trigger();
    const int slot = threadIdx.x >> 7, t = threadIdx.x & 127, warp = t >> 5, lane = t & 31;
    unsigned char* smem = attn_tc_smem + ((1024u - (smem_u32(attn_tc_smem) & 1023u)) & 1023u) + (size_t)slot * PF_SLOT_BYTES;
    unsigned char* Bs = smem;
    unsigned char* Qs = smem + 2 * PAGE_ATOM;
    unsigned char* Ps = Qs + PF_B_BYTES;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int i = 0; i < PF_SLOTS; ++i) { mbar_init(&bar_k[i], 1); mbar_init(&bar_v[i], 1); mbar_init(&bar_s[i], 1); mbar_init(&bar_o[i], 1); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(128u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *((volatile uint32_t*)&tmem_slot) + (uint32_t)(slot * PFN);
    const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
    volatile int* abortp = &abort_flag;
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(PFN >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
    const uint64_t pol = policy_evict_last();           // a page is read by every row tile behind it

    pdl_wait();

    auto load_page = [&](const CUtensorMap* map, uint64_t* bar, int seq, int c, int h) {
        const int row = layer_row0 + (page_table[seq * pages_per_seq + c] * H + h) * KV_PAGE;
        mbar_expect_tx(bar, 2 * PAGE_ATOM);
        tma_load_2d(Bs, map, 0, row, bar, pol);
        tma_load_2d(Bs + PAGE_ATOM, map, 64, row, bar, pol);
    };
    uint32_t n_k = 0, n_v = 0, n_s = 0, n_o = 0;        // completed uses of the slot's four barriers (their parities)
    uint32_t k_issued = 0, v_issued = 0;
    bool ok = true;
    // tile -> (head, 16 rows); tiles with the most pages first (they are the longest)
    for (int it = slot * gridDim.x + blockIdx.x; it < n_tiles * H && ok; it += gridDim.x * PF_SLOTS) {
        const int rt = n_tiles - 1 - it / H, h = it % H;
        const int r0 = rt * PFQ;
        const int pos_lo = row_pos[r0], pos_hi = row_pos[r0 + PFQ - 1], seq = row_seq[r0];
        const int n_pages = pos_hi / KV_PAGE + 1;
        if (t == 0) { load_page(&map_k, &bar_k[slot], seq, 0, h); ++k_issued; }
        // queries: operand row n is row n % 16 of the tile (hi term for n < 16, lo term after); 16-byte chunks
#pragma unroll
        for (int u = 0; u < (PFN * 16) / 128; ++u) {
            const int idx = t + u * 128, n = idx >> 4, c16 = idx & 15;
            const bf16* src = (n < PFQ ? q_hi : q_lo) + (size_t)(r0 + (n % PFQ)) * H * HD + (size_t)h * HD + c16 * 8;
            *(uint4*)(Qs + b_operand_offset<PFN>(n, c16 * 8)) = *(const uint4*)src;
        }
        fence_async_smem();
        slot_bar(slot);
        float l_thr[PFQ], o_acc[PFQ];
        float m_own = -CUDART_INF_F;                     // thread 8q: the running maximum of row q
#pragma unroll
        for (int q = 0; q < PFQ; ++q) { l_thr[q] = 0.0f; o_acc[q] = 0.0f; }
        for (int c = 0; c < n_pages && ok; ++c) {
            // ---- S^T = K . Q^T ----
            if (t == 0) {
                if (mbar_wait(&bar_k[slot], n_k & 1u, abortp)) {
                    tc_fence_after();
#pragma unroll
                    for (int k16 = 0; k16 < HD / 16; ++k16) {
                        const uint64_t adv = (uint64_t)((k16 & 3) * 2);
                        tc_mma_bf16(tmem_base, make_smem_desc(smem_u32(Bs + (k16 >> 2) * PAGE_ATOM)) + adv,
                                    make_smem_desc(smem_u32(Qs + (k16 >> 2) * (PFN * 128))) + adv, idesc, k16 > 0 ? 1u : 0u);
                    }
                    tc_commit(&bar_s[slot]);
                }
            }
            ++n_k;
            ok = mbar_wait(&bar_s[slot], n_s & 1u, abortp);
            ++n_s;
            if (!ok) break;
            tc_fence_after();
            if (t == 0) { load_page(&map_v, &bar_v[slot], seq, c, h); ++v_issued; }     // the first product is done with the page buffer
            float s[PFQ];
            {
                float v[PFN];
                tc_ld16(lane_base, v);
                tc_ld16(lane_base + 16u, v + 16);
#pragma unroll
                for (int q = 0; q < PFQ; ++q) s[q] = v[q] + v[PFQ + q];
            }
            // The page's maxima per row: the scores go through shared memory (the P operand's buffer, free until the
            // weights are written), transposed so that the eight threads 8q..8q+7 fold row q's 128 keys (16 each, then
            // three shuffles) instead of every thread folding all 16 rows across its warp.  Thread 8q owns row q's
            // running maximum: it raises it and leaves the new maximum and the rescaling factor of the row's older sums
            // in shared memory for everybody.  Words of a row are XOR-ed with 8 * (q & 3): no bank conflicts either way.
            const int key = c * KV_PAGE + t;
            float* sc = (float*)Ps;
#pragma unroll
            for (int q = 0; q < PFQ; ++q) {
                if (key > pos_lo + q) s[q] = -CUDART_INF_F;
                sc[q * KV_PAGE + (t ^ ((q & 3) * 8))] = s[q];
            }
            tc_fence_before();
            slot_bar(slot);
            {
                const int q = t >> 3, j = t & 7;
                float mx = -CUDART_INF_F;
#pragma unroll
                for (int i = 0; i < KV_PAGE / 8; ++i) mx = fmaxf(mx, sc[q * KV_PAGE + ((j + 8 * i) ^ ((q & 3) * 8))]);
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
                if (j == 0) {
                    const float m_new = fmaxf(m_own, mx);
                    const bool none = (m_new == -CUDART_INF_F);
                    row_ms[slot][q] = make_float2(m_new, (none || m_own == -CUDART_INF_F) ? 0.0f : exp2f(m_own - m_new));
                    m_own = m_new;
                }
            }
            slot_bar(slot);
            float scale[PFQ];
#pragma unroll
            for (int q = 0; q < PFQ; ++q) {
                const float2 ms = row_ms[slot][q];
                scale[q] = ms.y;
                const float pw = (ms.x == -CUDART_INF_F) ? 0.0f : exp2f(s[q] - ms.x);
                const bf16 hh = __float2bfloat16_rn(pw);
                const bf16 ll = __float2bfloat16_rn(pw - __bfloat162float(hh));
                *(bf16*)(Ps + b_operand_offset<PFN>(q, t)) = hh;
                *(bf16*)(Ps + b_operand_offset<PFN>(PFQ + q, t)) = ll;
                l_thr[q] = fmaf(l_thr[q], scale[q], pw);
            }
            fence_async_smem();
            slot_bar(slot);
            // ---- O^T = V^T . P^T ----
            if (t == 0) {
                if (mbar_wait(&bar_v[slot], n_v & 1u, abortp)) {
                    tc_fence_after();
#pragma unroll
                    for (int k16 = 0; k16 < KV_PAGE / 16; ++k16) {
                        const uint64_t adv = (uint64_t)((k16 & 3) * 2);
                        tc_mma_bf16(tmem_base, make_smem_desc(smem_u32(Bs + (k16 >> 2) * PAGE_ATOM)) + adv,
                                    make_smem_desc(smem_u32(Ps + (k16 >> 2) * (PFN * 128))) + adv, idesc, k16 > 0 ? 1u : 0u);
                    }
                    tc_commit(&bar_o[slot]);
                }
            }
            ++n_v;
            ok = mbar_wait(&bar_o[slot], n_o & 1u, abortp);
            ++n_o;
            if (!ok) break;
            tc_fence_after();
            if (c + 1 < n_pages && t == 0) { load_page(&map_k, &bar_k[slot], seq, c + 1, h); ++k_issued; }   // the second product is done with the buffer
            {
                float v[PFN];
                tc_ld16(lane_base, v);
                tc_ld16(lane_base + 16u, v + 16);
#pragma unroll
                for (int q = 0; q < PFQ; ++q) o_acc[q] = fmaf(o_acc[q], scale[q], v[q] + v[PFQ + q]);
            }
            tc_fence_before();
            slot_bar(slot);                              // the next first product overwrites the columns just read
        }
        if (!ok) break;
        // the weights' sums over all keys: within a warp, then the four warps in order
#pragma unroll
        for (int q = 0; q < PFQ; ++q) {
            float sum = l_thr[q];
            for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            if (lane == 0) red_sum[slot][warp][q] = sum;
        }
        slot_bar(slot);
#pragma unroll
        for (int q = 0; q < PFQ; ++q) {
            const float L = (red_sum[slot][0][q] + red_sum[slot][1][q]) + (red_sum[slot][2][q] + red_sum[slot][3][q]);
            const float o = o_acc[q] / L;
            const bf16 hh = __float2bfloat16_rn(o);
            const bf16 ll = __float2bfloat16_rn(o - __bfloat162float(hh));
            const size_t out = (size_t)(r0 + q) * H * HD + (size_t)h * HD + t;
            ao_hi[out] = hh;
            ao_lo[out] = ll;
        }
        slot_bar(slot);                                  // the staging buffers and the reduction scratch are free again
    }
    if (t == 0 && abort_flag) {
        if (k_issued) for (unsigned spin = 0; spin < WAIT_LIMIT && !mbar_try_wait(&bar_k[slot], (k_issued - 1) & 1u); ++spin) {}
        if (v_issued) for (unsigned spin = 0; spin < WAIT_LIMIT && !mbar_try_wait(&bar_v[slot], (v_issued - 1) & 1u); ++spin) {}
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicExch(err, ATTN_ERR_TIMEOUT);
    if (threadIdx.x < 32) {
        tc_fence_after();
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(*((volatile uint32_t*)&tmem_slot)), "r"(128u) : "memory");
    }
}

template <int G, int S>
anpd_status launch_attn_tc(anpd_model* m, anpd_kv* kv, int layer, int rows, int chunks, bool tree) {
    typedef AttnCfg<G, S> Cfg;
    const anpd_model_config& c = m->cfg;
    Workspace& ws = kv->ws;
    static bool attr_set[64] = {false};
    if (first_call_on_device(attr_set)) {
        CUDA_TRY(cudaFuncSetAttribute(attn_tc_kernel<G, S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::SMEM));
    }
    const int layer_row0 = layer * kv->total_pages * c.n_kv_heads * KV_PAGE;
    const int n_items = chunks * c.n_kv_heads * (rows / ANPD_ROWS);
    const int grid = std::min(m->num_sms, n_items);
    LAUNCH(&m->prof, m->stream, KC_ATTN, 0,
           (launch_k(attn_tc_kernel<G, S>, grid, Cfg::THREADS, Cfg::SMEM, m->stream, kv->map_k, kv->map_v, ws.q_hi, ws.q_lo, kv->page_table,
                     kv->pages_per_seq, ws.row_pos, ws.row_seq, c.n_q_heads, c.n_kv_heads, layer_row0, chunks, n_items, ws.attn_m,
                     ws.attn_l, ws.attn_o, ws.gemm_err, tree ? ws.row_slot : (const int*)nullptr,
                     tree ? ws.row_hole_lo : (const int*)nullptr, tree ? ws.row_hole_hi : (const int*)nullptr)));
    return ANPD_OK;
}

}  // namespace

// Attention of a prompt pass, straight to the O projection's input (no page partials, no merge).  rows: a multiple of 8; the
// row plan must cover the padding up to a multiple of 16.
anpd_status attn_prompt_enqueue(anpd_model* m, anpd_kv* kv, int layer, int rows) {
    const anpd_model_config& c = m->cfg;
    Workspace& ws = kv->ws;
    static bool attr_set[64] = {false};
    if (first_call_on_device(attr_set)) {
        CUDA_TRY(cudaFuncSetAttribute(attn_prompt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PF_SMEM));
    }
    const int layer_row0 = layer * kv->total_pages * c.n_kv_heads * KV_PAGE;
    const int n_tiles = (rows + PFQ - 1) / PFQ;
    const int grid = std::min(m->num_sms, (n_tiles * c.n_q_heads + PF_SLOTS - 1) / PF_SLOTS);
    LAUNCH(&m->prof, m->stream, KC_ATTN, 0,
           (launch_k(attn_prompt_kernel, grid, PF_SLOTS * 128, PF_SMEM, m->stream, kv->map_k, kv->map_v, ws.q_hi, ws.q_lo, kv->page_table,
                     kv->pages_per_seq, ws.row_pos, ws.row_seq, c.n_q_heads, layer_row0, n_tiles, ws.ao_hi, ws.ao_lo, ws.gemm_err)));
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}

anpd_status attn_tc_enqueue(anpd_model* m, anpd_kv* kv, int layer, int rows, int max_pos, bool tree) {
    const int chunks = max_pos / KV_PAGE + 1;
    const int n_items = chunks * m->cfg.n_kv_heads * (rows / ANPD_ROWS);
    switch (m->cfg.n_q_heads / m->cfg.n_kv_heads) {
        // one query head per kv head fits five slots; while every item finds a slot with four, four are faster
        // (measured at the 7B shape: 1.2 % of the step at 17 pages; with 33 pages five slots win by 2.4 %)
        case 1: return n_items <= 4 * m->num_sms ? launch_attn_tc<1, 4>(m, kv, layer, rows, chunks, tree)
                                                 : launch_attn_tc<1, 5>(m, kv, layer, rows, chunks, tree);
        case 2: return launch_attn_tc<2, 4>(m, kv, layer, rows, chunks, tree);
        case 4: return launch_attn_tc<4, 3>(m, kv, layer, rows, chunks, tree);
        case 8: return launch_attn_tc<8, 2>(m, kv, layer, rows, chunks, tree);
    }
    return ANPD_ERR_ARG;
}
