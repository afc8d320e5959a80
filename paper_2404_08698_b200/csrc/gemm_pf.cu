// Projection GEMM for prompt passes (Algorithm 1's LLM(prompt)): hundreds to thousands of rows at once, so the product is
// bound by the tensor cores, not by reading the weights:  out[row][n] = sum_k W[n][k] * (a_hi[row][k] + a_lo[row][k]).
//
// A CTA owns an output tile of 256 features x 256 rows and walks the whole contraction dimension.  Per 64-wide k-block it
// brings two 128-feature weight blocks (the same pre-swizzled 16 KB blocks the decode GEMM streams, any block is addressable
// through gemm_block_slot) and the 256 rows' hi and lo activation tiles (four TMA boxes of 128 rows) into shared memory -
// 96 KB for sixteen 128 x 256 x 16 MMAs - and accumulates W0 x hi, W0 x lo into one 256-column accumulator in tensor
// memory and W1 x hi, W1 x lo into a second one: every activation byte is used against 256 features, every weight byte
// against 256 rows.  Tiles that share a weight pair run on neighbouring CTAs at the same time, so a weight block crosses HBM
// once per prompt pass and is served from L2 otherwise.  A projection with fewer tiles than would keep every SM busy is also cut
// along K into `ksplit` equal parts (the same cut for every tile): part s leaves its sums in partial-sum slab s and the
// consumers add the slabs in order, as they add the decode GEMM's segments.  A projection whose tiles fill some rounds of
// CTAs and a fraction of one more has the tiles of that last round alone cut into 2 or 3 parts, so that the round takes a
// half or a third of a tile's time on all SMs instead of a whole tile's time on some.
#include "internal.h"
#include "tc_ptx.cuh"

#include <algorithm>
#include <vector>

typedef __nv_bfloat16 bf16;

namespace {

using namespace tc;

constexpr int PF_TILE_TOK = 256;
constexpr int PF_THREADS = 192;          // warp 0: producer, warp 1: MMA issuer + tensor-memory owner, warps 2-5: epilogue
constexpr int PF_BLOCK = 16384;          // one 128 x 64 bf16 operand tile
constexpr int PF_STAGE = 6 * PF_BLOCK;   // W0, W1, hi rows 0-127, hi rows 128-255, lo rows 0-127, lo rows 128-255
constexpr int PF_STAGES = 2;
constexpr int PF_ERR_TIMEOUT = 205;

struct PfArgs {
    float* out; int ld;
    int N, rows;
    int m_tiles, k_blocks, n_ft, n_tt, ksplit;
    int tail_from, tail_split;         // output tiles from tail_from on are cut into tail_split parts instead of ksplit
    size_t seg_stride;                 // elements between the partial-sum slabs of two K parts
    long long total; int G;
    int* err;
};

// work item -> (output tile, K part, parts of that tile); K part fastest
__device__ __forceinline__ void pf_item(const PfArgs& g, int item, int& ot, int& ks, int& parts) {
    const int uniform = g.tail_from * g.ksplit;
    if (item < uniform) { ot = item / g.ksplit; ks = item - ot * g.ksplit; parts = g.ksplit; }
    else { const int j = item - uniform; ot = g.tail_from + j / g.tail_split; ks = j % g.tail_split; parts = g.tail_split; }
}

__global__ void __launch_bounds__(PF_THREADS, 1)
gemm_pf_kernel(const bf16* __restrict__ w_blocks, const __grid_constant__ CUtensorMap map_hi, const __grid_constant__ CUtensorMap map_lo,
               const PfArgs g) {
    extern __shared__ __align__(1024) unsigned char pf_smem_raw[];
    __shared__ uint64_t bar_full[PF_STAGES], bar_empty[PF_STAGES], bar_acc_full, bar_acc_empty;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    pdl_trigger();
    unsigned char* smem = pf_smem_raw + ((1024u - (smem_u32(pf_smem_raw) & 1023u)) & 1023u);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = g.tail_from * g.ksplit + (g.n_ft * g.n_tt - g.tail_from) * g.tail_split;     // work items

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < PF_STAGES; ++s) { mbar_init(&bar_full[s], 1); mbar_init(&bar_empty[s], 1); }
        mbar_init(&bar_acc_full, 1); mbar_init(&bar_acc_empty, 4);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *((volatile uint32_t*)&tmem_slot);
    volatile int* abortp = &abort_flag;

    pdl_wait();                                        // the activations come from the kernel before

    if (warp == 0) {
        if (lane == 0) {
            const uint64_t pol_w = policy_evict_last(), pol_a = policy_evict_last();    // both are re-read by other CTAs: keep them in L2
            int stage = 0;
            uint32_t phase = 0;
            long long issued = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
                int ot, ks, parts;
                pf_item(g, tile, ot, ks, parts);
                const int ft = ot / g.n_tt, tt = ot - ft * g.n_tt;
                const int t0 = 2 * ft, t1 = min(2 * ft + 1, g.m_tiles - 1);      // an odd tile count: the last pair repeats its tile
                const int row0 = tt * PF_TILE_TOK;
                const int kb_end = (int)((long long)(ks + 1) * g.k_blocks / parts);
                for (int kb = (int)((long long)ks * g.k_blocks / parts); kb < kb_end; ++kb) {
                    ok = mbar_wait(&bar_empty[stage], phase ^ 1u, abortp);
                    if (!ok) break;
                    unsigned char* st = smem + (size_t)stage * PF_STAGE;
                    mbar_expect_tx(&bar_full[stage], (uint32_t)PF_STAGE);
                    bulk_load(st, w_blocks + (size_t)gemm_block_slot((long long)t0 * g.k_blocks + kb, g.total, g.G) * (128 * 64), PF_BLOCK, &bar_full[stage], pol_w);
                    bulk_load(st + PF_BLOCK, w_blocks + (size_t)gemm_block_slot((long long)t1 * g.k_blocks + kb, g.total, g.G) * (128 * 64), PF_BLOCK, &bar_full[stage], pol_w);
                    tma_load_2d(st + 2 * PF_BLOCK, &map_hi, kb * 64, row0, &bar_full[stage], pol_a);
                    tma_load_2d(st + 3 * PF_BLOCK, &map_hi, kb * 64, row0 + 128, &bar_full[stage], pol_a);
                    tma_load_2d(st + 4 * PF_BLOCK, &map_lo, kb * 64, row0, &bar_full[stage], pol_a);
                    tma_load_2d(st + 5 * PF_BLOCK, &map_lo, kb * 64, row0 + 128, &bar_full[stage], pol_a);
                    ++issued;
                    if (++stage == PF_STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // gave up: let every copy already issued land before the CTA may exit
                const long long n = issued < PF_STAGES ? issued : PF_STAGES;
                for (long long i = 0; i < n; ++i) {
                    const long long idx = issued - 1 - i;
                    const int s = (int)(idx % PF_STAGES);
                    const uint32_t ph = (uint32_t)((idx / PF_STAGES) & 1);
                    for (unsigned spin = 0; spin < WAIT_LIMIT && !mbar_try_wait(&bar_full[s], ph); ++spin) {}
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // fp32 accumulate, bf16 x bf16, both operands K-major, M = 128 (weight features), N = 256 (rows)
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
            int stage = 0;
            uint32_t phase = 0;
            int done_tiles = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++done_tiles) {
                ok = mbar_wait(&bar_acc_empty, (uint32_t)((done_tiles & 1) ^ 1), abortp);      // the epilogue has read the previous tile
                if (!ok) break;
                tc_fence_after();
                int ot, ks, parts;
                pf_item(g, tile, ot, ks, parts);
                const int kb_begin = (int)((long long)ks * g.k_blocks / parts), kb_end = (int)((long long)(ks + 1) * g.k_blocks / parts);
                for (int kb = kb_begin; kb < kb_end; ++kb) {
                    ok = mbar_wait(&bar_full[stage], phase, abortp);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sb = smem_u32(smem + (size_t)stage * PF_STAGE);
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const uint64_t dw = make_smem_desc(sb + j * PF_BLOCK);
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            const uint64_t da = make_smem_desc(sb + (2 + 2 * half) * PF_BLOCK);     // 256 rows: two boxes, one after the other
#pragma unroll
                            for (int k16 = 0; k16 < 4; ++k16) {
                                const uint64_t adv = (uint64_t)(k16 * 2);
                                tc_mma_bf16(tmem_base + (uint32_t)(j * 256), dw + adv, da + adv, idesc, ((kb - kb_begin) | half | k16) ? 1u : 0u);
                            }
                        }
                    }
                    tc_commit(&bar_empty[stage]);
                    if (++stage == PF_STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_commit(&bar_acc_full);
            }
        }
    } else {
        const int quad = warp & 3;
        int done_tiles = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++done_tiles) {
            int ot, ks, parts;
            pf_item(g, tile, ot, ks, parts);
            const int ft = ot / g.n_tt, tt = ot - ft * g.n_tt;
            ok = mbar_wait(&bar_acc_full, (uint32_t)(done_tiles & 1), abortp);
            if (!ok) break;
            tc_fence_after();
            const int row0 = tt * PF_TILE_TOK;
#pragma unroll 1
            for (int j = 0; j < 2; ++j) {
                const int t = 2 * ft + j;
                if (t >= g.m_tiles) break;
                const int n = t * 128 + quad * 32 + lane;
#pragma unroll 1
                for (int c0 = 0; c0 < PF_TILE_TOK; c0 += 16) {
                    if (row0 + c0 >= g.rows) break;
                    float v[16];
                    tc_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(j * 256 + c0), v);
                    if (n < g.N) {
                        float* out = g.out + (size_t)ks * g.seg_stride + (size_t)(row0 + c0) * g.ld + n;
#pragma unroll
                        for (int r = 0; r < 16; ++r)
                            if (row0 + c0 + r < g.rows) out[(size_t)r * g.ld] = v[r];
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_acc_empty);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
    if (threadIdx.x == 0 && abort_flag) atomicExch(g.err, PF_ERR_TIMEOUT);
}

}  // namespace

// Steps on the busiest CTA when the work items go to the CTAs round robin (a tile's epilogue counts as about six steps).
static long long pf_cost(int n_ot, int k_blocks, int num_sms, const PfSchedule& s) {
    const int uniform = s.tail_from * s.ksplit;
    const int n_items = uniform + (n_ot - s.tail_from) * s.tail_split;
    const int grid = std::min(num_sms, n_items);
    std::vector<long long> load((size_t)grid, 0);
    for (int it = 0; it < n_items; ++it) {
        const int parts = it < uniform ? s.ksplit : s.tail_split;
        load[(size_t)(it % grid)] += (k_blocks + parts - 1) / parts + 6;
    }
    return *std::max_element(load.begin(), load.end());
}

// The cut along K with the fewest steps on the busiest SM: every tile in 1, 2 or 3 parts, or the tiles of the last, partly
// filled round alone in 2 or 3 parts.
PfSchedule gemm_pf_schedule(int n_ft, int n_tt, int k_blocks, int num_sms) {
    const int n_ot = n_ft * n_tt;
    PfSchedule best{1, n_ot, 1};
    long long best_cost = pf_cost(n_ot, k_blocks, num_sms, best);
    for (int s = 2; s <= 3; ++s) {
        const PfSchedule c{s, n_ot, 1};
        const long long cost = pf_cost(n_ot, k_blocks, num_sms, c);
        if (cost < best_cost) { best = c; best_cost = cost; }
    }
    const int full = n_ot / num_sms;
    if (full >= 1 && n_ot % num_sms != 0) {
        const int from = (full * num_sms / n_tt) * n_tt;            // whole feature pairs stay uncut
        for (int s = 2; s <= 3 && from > 0; ++s) {
            const PfSchedule c{1, from, s};
            const long long cost = pf_cost(n_ot, k_blocks, num_sms, c);
            if (cost < best_cost) { best = c; best_cost = cost; }
        }
    }
    return best;
}

anpd_status gemm_pf_enqueue(const GemmPlan& plan, const bf16* w_blocks, const CUtensorMap& map_hi, const CUtensorMap& map_lo, int rows,
                            float* out, int ld, size_t seg_stride, PfSchedule sched, int num_sms, int* err, cudaStream_t st, Profiler* prof) {
    constexpr int smem = PF_STAGES * PF_STAGE + 1024;
    static bool attr_set[64] = {false};
    if (first_call_on_device(attr_set)) {
        CUDA_TRY(cudaFuncSetAttribute(gemm_pf_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    }
    PfArgs g;
    g.out = out; g.ld = ld; g.N = plan.N; g.rows = rows;
    g.m_tiles = plan.m_tiles; g.k_blocks = plan.k_blocks;
    g.n_ft = (plan.m_tiles + 1) / 2;
    g.n_tt = (rows + PF_TILE_TOK - 1) / PF_TILE_TOK;
    g.total = (long long)plan.m_tiles * plan.k_blocks;
    g.G = plan.grid;
    g.ksplit = sched.ksplit; g.tail_from = sched.tail_from; g.tail_split = sched.tail_split; g.seg_stride = seg_stride;
    g.err = err;
    const int grid = std::min(num_sms, sched.tail_from * sched.ksplit + (g.n_ft * g.n_tt - sched.tail_from) * sched.tail_split);
    LAUNCH(prof, st, KC_GEMM, 2.0 * (double)plan.N * (double)plan.K,
           (launch_k(gemm_pf_kernel, grid, PF_THREADS, (size_t)smem, st, w_blocks, map_hi, map_lo, g)));
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}
