// Attention of the verify step for head dimension 128 on the sm_100a tensor cores
// (paper Section 3.1, "Verification": the K+1 rows of a step attend to the cached keys).
//
// One CTA handles one 128-key page of one kv head for one group of 8 rows.  With so few query rows
// the operands are swapped, as in the weight GEMM: the page is the MMA's 128-row M operand and the
// 8 x G query vectors that share the kv head are its N operand.
//   S^T [128 keys x N]  = K page   [128 keys x 128 dims] . Q^T     (tcgen05.mma, accumulator in tensor memory)
//   O^T [128 dims x N]  = V^T page [128 dims x 128 keys] . P^T
// K pages are stored [key][dim] and V pages transposed [dim][key], so both are K-major and arrive by
// TMA in the 128-byte-swizzled layout the MMA reads.  Queries and softmax weights enter as two bf16
// terms each (hi rows then lo rows of the N operand, N = 2 x 8 x G), so only the cache's own bf16
// rounding is left; the two halves of an accumulator are added when it is read back.
// Thread t of the CTA owns tensor-memory lane t: key t of the page after the first product, output
// dimension t after the second.  The softmax over the page's keys is a reduction across threads
// (shuffle tree inside a warp, then the four warps in warp order).  Each page leaves a partial
// (max, sum, weighted values) per query vector; the combine kernel merges pages in page order.
// Every value depends on the row's own position and inputs only: masked keys contribute exact zeros
// and the order of every sum is fixed by key positions, so a row's result does not depend on which
// other rows share the launch.
#include "internal.h"
#include "tc_ptx.cuh"

#include <math_constants.h>

typedef __nv_bfloat16 bf16;

namespace {

using namespace tc;

constexpr int HD = 128;
constexpr int PAGE_ATOM = 128 * 128;        // bytes of a 128-row x 64-column bf16 tile (one TMA box)
constexpr int ATTN_TC_THREADS = 128;
constexpr int ATTN_ERR_TIMEOUT = 202;

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Byte offset of element (row n, column k) of an [N rows][128 columns] bf16 operand held as two
// 64-column tiles in the 128-byte-swizzled K-major layout (8-row groups 1024 bytes apart).
template <int N>
__device__ __forceinline__ int b_operand_offset(int n, int k) {
    const int kk = k & 63;
    return (k >> 6) * (N * 128) + (n >> 3) * 1024 + (n & 7) * 128 + ((((kk >> 3) ^ (n & 7))) << 4) + (kk & 7) * 2;
}

template <int G>
__global__ void __launch_bounds__(ATTN_TC_THREADS)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const bf16* __restrict__ q_hi,
               const bf16* __restrict__ q_lo, const int* __restrict__ page_table, int pages_per_seq, const int* __restrict__ row_pos,
               const int* __restrict__ row_seq, int Hq, int Hkv, int layer_row0, float* __restrict__ pm, float* __restrict__ pl,
               float* __restrict__ po, int* err) {
    constexpr int Q = 8 * G;                 // query vectors: 8 rows x G heads of the group
    constexpr int N = 2 * Q;                 // MMA N: hi terms then lo terms
    constexpr int B_BYTES = N * 256;         // one N-row operand (two 64-column tiles)
    constexpr int TMEM_COLS = (2 * N < 32) ? 32 : 2 * N;      // S^T in columns [0, N), O^T in [N, 2N)
    extern __shared__ __align__(1024) unsigned char attn_tc_smem[];
    __shared__ uint64_t bar_kv, bar_s, bar_o;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ float red[4][Q];

    pdl_trigger();
    unsigned char* smem = attn_tc_smem + ((1024u - (smem_u32(attn_tc_smem) & 1023u)) & 1023u);
    unsigned char* Ks = smem;                        // two tiles: dims 0..63, dims 64..127
    unsigned char* Vs = smem + 2 * PAGE_ATOM;        // two tiles: keys 0..63, keys 64..127
    unsigned char* Qs = smem + 4 * PAGE_ATOM;
    unsigned char* Ps = Qs + B_BYTES;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int c = blockIdx.x, kvh = blockIdx.y, r0 = blockIdx.z * ANPD_ROWS;

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(&bar_kv, 1); mbar_init(&bar_s, 1); mbar_init(&bar_o, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"((uint32_t)TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *((volatile uint32_t*)&tmem_slot);
    volatile int* abortp = &abort_flag;

    pdl_wait();                                      // the row plan, the queries and this step's K/V rows come from earlier kernels
    const int pos_lo = row_pos[r0], pos_hi = row_pos[r0 + ANPD_ROWS - 1];
    const bool active = c * KV_PAGE <= pos_hi;       // block-uniform: pages beyond the last row's position hold nothing any row may see
    bool ok = true;
    // fp32 accumulate, bf16 x bf16, both operands K-major, M = 128
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
    if (active) {
        if (tid == 0) {
            const int page = page_table[row_seq[r0] * pages_per_seq + c];
            const int row = layer_row0 + (page * Hkv + kvh) * KV_PAGE;       // first row of the page in the pools' 2-D view
            const uint64_t pol = policy_evict_first();
            mbar_expect_tx(&bar_kv, 4 * PAGE_ATOM);
            tma_load_2d(Ks, &map_k, 0, row, &bar_kv, pol);
            tma_load_2d(Ks + PAGE_ATOM, &map_k, 64, row, &bar_kv, pol);
            tma_load_2d(Vs, &map_v, 0, row, &bar_kv, pol);
            tma_load_2d(Vs + PAGE_ATOM, &map_v, 64, row, &bar_kv, pol);
        }
        // queries: row n of the operand is query vector n % Q (hi term for n < Q, lo term after); 16-byte chunks
        for (int idx = tid; idx < N * 16; idx += ATTN_TC_THREADS) {
            const int n = idx >> 4, c16 = idx & 15;
            const int qn = n % Q, g = qn >> 3, r = qn & 7;
            const bf16* src = (n < Q ? q_hi : q_lo) + (size_t)(r0 + r) * Hq * HD + (size_t)(kvh * G + g) * HD + c16 * 8;
            *(uint4*)(Qs + b_operand_offset<N>(n, c16 * 8)) = *(const uint4*)src;
        }
        fence_async_smem();
        __syncthreads();

        if (tid == 0) {
            ok = mbar_wait(&bar_kv, 0, abortp);
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int k16 = 0; k16 < HD / 16; ++k16) {
                    const uint64_t adv = (uint64_t)((k16 & 3) * 2);                 // 32 bytes along K inside the swizzle row, 16-byte units
                    tc_mma_bf16(tmem_base, make_smem_desc(smem_u32(Ks + (k16 >> 2) * PAGE_ATOM)) + adv,
                                make_smem_desc(smem_u32(Qs + (k16 >> 2) * (N * 128))) + adv, idesc, k16 > 0 ? 1u : 0u);
                }
                tc_commit(&bar_s);
            }
        }
        ok = mbar_wait(&bar_s, 0, abortp) && ok;
        ok = __syncthreads_and(ok) != 0;
    }
    if (active && ok) {
        tc_fence_after();
        const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
        float s[Q];
        {
            float v[N];
#pragma unroll
            for (int c0 = 0; c0 < N; c0 += 16) tc_ld16(lane_base + (uint32_t)c0, v + c0);
#pragma unroll
            for (int q = 0; q < Q; ++q) s[q] = v[q] + v[Q + q];
        }
        // mask by position (this thread's key is c * 128 + tid), maximum over the page's keys per query vector
        const int key = c * KV_PAGE + tid;
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            if (key > pos_lo + (q & 7)) s[q] = -CUDART_INF_F;
            float mx = s[q];
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            if (lane == 0) red[warp][q] = mx;
        }
        __syncthreads();
        float m[Q];
#pragma unroll
        for (int q = 0; q < Q; ++q) m[q] = fmaxf(fmaxf(red[0][q], red[1][q]), fmaxf(red[2][q], red[3][q]));
        __syncthreads();
        // weights (base-2 domain: the queries carry log2(e) / sqrt(hd)), their sum, and the P operand
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            const float p = (m[q] == -CUDART_INF_F) ? 0.0f : exp2f(s[q] - m[q]);
            const bf16 h = __float2bfloat16_rn(p);
            const bf16 l = __float2bfloat16_rn(p - __bfloat162float(h));
            *(bf16*)(Ps + b_operand_offset<N>(q, tid)) = h;
            *(bf16*)(Ps + b_operand_offset<N>(Q + q, tid)) = l;
            float sum = p;
            for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            if (lane == 0) red[warp][q] = sum;
        }
        fence_async_smem();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after();
#pragma unroll
            for (int k16 = 0; k16 < KV_PAGE / 16; ++k16) {
                const uint64_t adv = (uint64_t)((k16 & 3) * 2);
                tc_mma_bf16(tmem_base + (uint32_t)N, make_smem_desc(smem_u32(Vs + (k16 >> 2) * PAGE_ATOM)) + adv,
                            make_smem_desc(smem_u32(Ps + (k16 >> 2) * (N * 128))) + adv, idesc, k16 > 0 ? 1u : 0u);
            }
            tc_commit(&bar_o);
        }
        if (tid < Q) {
            const int q = tid;
            const size_t out = ((size_t)(r0 + (q & 7)) * Hq + (kvh * G + (q >> 3))) * pages_per_seq + c;
            pm[out] = m[q];
            pl[out] = (red[0][q] + red[1][q]) + (red[2][q] + red[3][q]);
        }
        ok = mbar_wait(&bar_o, 0, abortp);
        if (ok) {
            tc_fence_after();
            float v[N];
#pragma unroll
            for (int c0 = 0; c0 < N; c0 += 16) tc_ld16(lane_base + (uint32_t)(N + c0), v + c0);
#pragma unroll
            for (int q = 0; q < Q; ++q) {
                const size_t out = ((size_t)(r0 + (q & 7)) * Hq + (kvh * G + (q >> 3))) * pages_per_seq + c;
                po[out * HD + tid] = v[q] + v[Q + q];
            }
        }
    }
    if (active && tid == 0 && abort_flag) {
        // gave up somewhere: let the page copies land before the CTA may exit
        for (unsigned spin = 0; spin < WAIT_LIMIT && !mbar_try_wait(&bar_kv, 0); ++spin) {}
        atomicExch(err, ATTN_ERR_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

template <int G>
anpd_status launch_attn_tc(anpd_model* m, anpd_kv* kv, int layer, int rows, int chunks) {
    const anpd_model_config& c = m->cfg;
    Workspace& ws = kv->ws;
    constexpr int N = 16 * G;
    const size_t smem = 4 * PAGE_ATOM + 2 * (size_t)N * 256 + 1024;
    static bool attr_set = false;
    if (!attr_set) {
        CUDA_TRY(cudaFuncSetAttribute(attn_tc_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr_set = true;
    }
    const int layer_row0 = layer * kv->total_pages * c.n_kv_heads * KV_PAGE;
    dim3 grid(chunks, c.n_kv_heads, rows / ANPD_ROWS);
    LAUNCH(&m->prof, m->stream, KC_ATTN, 0,
           (launch_k(attn_tc_kernel<G>, grid, ATTN_TC_THREADS, smem, m->stream, kv->map_k, kv->map_v, ws.q_hi, ws.q_lo, kv->page_table,
                     kv->pages_per_seq, ws.row_pos, ws.row_seq, c.n_q_heads, c.n_kv_heads, layer_row0, ws.attn_m, ws.attn_l, ws.attn_o,
                     ws.gemm_err)));
    return ANPD_OK;
}

}  // namespace

anpd_status attn_tc_enqueue(anpd_model* m, anpd_kv* kv, int layer, int rows, int max_pos) {
    const int chunks = max_pos / KV_PAGE + 1;
    switch (m->cfg.n_q_heads / m->cfg.n_kv_heads) {
        case 1: return launch_attn_tc<1>(m, kv, layer, rows, chunks);
        case 2: return launch_attn_tc<2>(m, kv, layer, rows, chunks);
        case 4: return launch_attn_tc<4>(m, kv, layer, rows, chunks);
        case 8: return launch_attn_tc<8>(m, kv, layer, rows, chunks);
    }
    return ANPD_ERR_ARG;
}
