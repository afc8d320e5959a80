// Weight-streaming GEMM for the verify forward on sm_100a:  part[seg][row][n] = sum_k W[n][k] * (a_hi[row][k] + a_lo[row][k])
//
// The step's K+1 <= 8 rows (x batch) are far too few to fill the tensor core's M side, so the
// operands are swapped: a 128-row tile of the weight matrix is the MMA's M operand, the rows of
// the step are its N operand (padded to a multiple of 16), and the accumulator D[128 x NB] lives
// in tensor memory.  The kernel is bound by reading W from HBM exactly once:
//   - one persistent CTA per SM; the (m_tile, k_block) grid is cut into equal contiguous ranges
//     ("stream-K"), so every SM streams the same number of bytes whatever the matrix shape;
//   - a producer thread keeps a ring of TMA loads (128x64 bf16 weight tile + the two activation
//     tiles) in flight through mbarriers; an MMA thread issues tcgen05.mma straight from shared
//     memory; four epilogue warps drain finished accumulators from tensor memory while the next
//     segment is already accumulating in the other half (double-buffered TMEM);
//   - a range that covers only part of a tile's K extent writes a partial sum; the consumers of
//     the GEMM add a tile's partial sums in ascending K order, a fixed order that depends on the
//     matrix shape only - never on the number of rows - so results are bit-reproducible and
//     identical for greedy and draft-verify steps.
// Activations arrive as two bf16 terms (hi + lo) and both are multiplied with the same weight
// tile, which keeps fp32-class activation precision on a bf16 tensor core at no extra HBM cost.
#include "internal.h"
#include "tc_ptx.cuh"

#include <cuda.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>

typedef __nv_bfloat16 bf16;

namespace {

using namespace tc;

constexpr int TILE_M = 128;             // weight rows per tile (MMA M)
constexpr int TILE_K = 64;              // bf16 elements per k-block = one 128-byte swizzle row
constexpr int A_BYTES = TILE_M * TILE_K * 2;
constexpr int GEMM_THREADS = 192;       // warp 0: TMA producer, warp 1: MMA issuer + TMEM owner, warps 2-5: epilogue
constexpr int MAX_STAGES = 12;
constexpr int RING_STAGES = 5;
constexpr int GEMM_ERR_TIMEOUT = 201;

struct GemmArgs {
    float* part;            // [segments][rows_ld][ld_part]
    size_t seg_stride;      // elements between segment slabs
    int ld_part;
    int N, rows;            // valid output features / valid rows (stores are clipped to these)
    int NB;                 // MMA N: rows padded to a multiple of 16
    int m_tiles, k_blocks;
    int stages;
    int tmem_cols;          // power of two >= 4 * NB (two accumulators of 2 * NB columns: W x hi and W x lo side by side)
    const int* first_cta;   // [m_tiles] CTA that owns the first k-block of a tile
    int* err;
};

__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tc_kernel(const bf16* __restrict__ w_blocks, const __grid_constant__ CUtensorMap map_hi,
               const __grid_constant__ CUtensorMap map_lo, const GemmArgs g) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ uint64_t bar_full[MAX_STAGES], bar_empty[MAX_STAGES], bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    // the swizzled tiles need 1024-byte alignment in the shared address space
    pdl_trigger();
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int stage_bytes = A_BYTES + 2 * g.NB * 128;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // this CTA's contiguous range of (m_tile, k_block) pairs
    const long long total = (long long)g.m_tiles * g.k_blocks;
    const long long lo = (long long)blockIdx.x * total / gridDim.x, hi = (long long)(blockIdx.x + 1) * total / gridDim.x;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < g.stages; ++s) { mbar_init(&bar_full[s], 1); mbar_init(&bar_empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&bar_acc_full[b], 1); mbar_init(&bar_acc_empty[b], 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"((uint32_t)g.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *((volatile uint32_t*)&tmem_base_slot);
    volatile int* abortp = &abort_flag;

    if (warp == 0) {
        // ---------------- producer ----------------
        if (lane == 0) {
            const uint64_t pol_w = policy_evict_first(), pol_a = policy_evict_last();
            int stage = 0;
            uint32_t phase = 0;
            long long issued = 0;
            bool ok = true;
            // The weights do not depend on the previous kernel: request the first ring of weight tiles at
            // once, and only then wait for the kernel that produces this GEMM's activations.
            const long long ahead = min((long long)g.stages, hi - lo);
            for (long long i = 0; i < ahead; ++i) {
                unsigned char* sa = smem + (size_t)i * stage_bytes;
                mbar_expect_tx(&bar_full[i], (uint32_t)stage_bytes);
                bulk_load(sa, w_blocks + (size_t)(i * gridDim.x + blockIdx.x) * (TILE_M * TILE_K), A_BYTES, &bar_full[i], pol_w);
            }
            pdl_wait();
            int kb = (int)(lo % g.k_blocks);            // k-block of the next activation load; advanced without divisions
            for (long long i = 0; i < ahead; ++i) {
                unsigned char* sa = smem + (size_t)i * stage_bytes;
                tma_load_2d(sa + A_BYTES, &map_hi, kb * TILE_K, 0, &bar_full[i], pol_a);
                tma_load_2d(sa + A_BYTES + g.NB * 128, &map_lo, kb * TILE_K, 0, &bar_full[i], pol_a);
                if (++kb == g.k_blocks) kb = 0;
            }
            issued = ahead;
            stage = (int)(ahead % g.stages);
            phase = (ahead == g.stages) ? 1u : 0u;
            for (long long blk = lo + ahead; blk < hi && ok; ++blk) {
                ok = mbar_wait(&bar_empty[stage], phase ^ 1u, abortp);
                if (!ok) break;
                unsigned char* sa = smem + (size_t)stage * stage_bytes;
                mbar_expect_tx(&bar_full[stage], (uint32_t)stage_bytes);
                bulk_load(sa, w_blocks + (size_t)((blk - lo) * gridDim.x + blockIdx.x) * (TILE_M * TILE_K), A_BYTES, &bar_full[stage], pol_w);   // this CTA's slot of the step's window
                tma_load_2d(sa + A_BYTES, &map_hi, kb * TILE_K, 0, &bar_full[stage], pol_a);
                tma_load_2d(sa + A_BYTES + g.NB * 128, &map_lo, kb * TILE_K, 0, &bar_full[stage], pol_a);
                if (++kb == g.k_blocks) kb = 0;
                ++issued;
                if (++stage == g.stages) { stage = 0; phase ^= 1u; }
            }
            if (!ok) {
                // gave up: let every copy already issued land before the CTA may exit
                const long long n = issued < g.stages ? issued : g.stages;
                for (long long i = 0; i < n; ++i) {
                    const long long idx = issued - 1 - i;
                    const int s = (int)(idx % g.stages);
                    const uint32_t ph = (uint32_t)((idx / g.stages) & 1);
                    for (unsigned spin = 0; spin < WAIT_LIMIT && !mbar_try_wait(&bar_full[s], ph); ++spin) {}
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        pdl_wait();
        if (lane == 0) {
            // fp32 accumulate, bf16 x bf16, both operands K-major, N = 2 * NB (hi rows then lo rows), M = 128
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)((2 * g.NB) >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);
            int stage = 0;
            uint32_t phase = 0;
            int seg = 0;
            bool ok = true;
            long long blk = lo;
            while (blk < hi && ok) {
                const int tile = (int)(blk / g.k_blocks);
                const long long seg_end = min(hi, (long long)(tile + 1) * g.k_blocks);
                const int buf = seg & 1;
                ok = mbar_wait(&bar_acc_empty[buf], (uint32_t)(((seg >> 1) & 1) ^ 1), abortp);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * 2 * g.NB);
                uint32_t acc = 0;
                for (; blk < seg_end; ++blk) {
                    ok = mbar_wait(&bar_full[stage], phase, abortp);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem + (size_t)stage * stage_bytes);
                    // the lo rows follow the hi rows in the stage, so one descriptor spans both: one MMA reads the
                    // weight slice from shared memory once and yields W x hi in columns [0, NB) and W x lo in [NB, 2 NB)
                    const uint64_t da = make_smem_desc(sa), db = make_smem_desc(sa + A_BYTES);
#pragma unroll
                    for (int k16 = 0; k16 < TILE_K / 16; ++k16) {
                        const uint64_t adv = (uint64_t)(k16 * 32 >> 4);     // 16 bf16 = 32 bytes along K inside the swizzle row
                        tc_mma_bf16(d_tmem, da + adv, db + adv, idesc, acc);
                        acc = 1;
                    }
                    tc_commit(&bar_empty[stage]);        // frees the stage once these MMAs have read it
                    if (++stage == g.stages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_commit(&bar_acc_full[buf]);           // accumulator complete
                ++seg;
            }
        }
    } else {
        // ---------------- epilogue: TMEM -> registers -> partial sums in global memory ----------------
        pdl_wait();                                       // the partial-sum buffer may still be read by the previous kernel
        const int quad = warp & 3;                        // a warp may only touch TMEM lanes 32*(warp%4)..+31
        int seg = 0;
        bool ok = true;
        long long blk = lo;
        while (blk < hi && ok) {
            const int tile = (int)(blk / g.k_blocks);
            const long long seg_end = min(hi, (long long)(tile + 1) * g.k_blocks);
            const int buf = seg & 1;
            ok = mbar_wait(&bar_acc_full[buf], (uint32_t)((seg >> 1) & 1), abortp);
            if (!ok) break;
            tc_fence_after();
            const int ordinal = (int)blockIdx.x - g.first_cta[tile];      // position of this segment in the tile's K order
            const int n = tile * TILE_M + quad * 32 + lane;
            float* out = g.part + (size_t)ordinal * g.seg_stride + n;
            for (int c0 = 0; c0 < g.NB; c0 += 16) {
                float v[16], w[16];
                tc_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * 2 * g.NB + c0), v);
                tc_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * 2 * g.NB + g.NB + c0), w);
                if (n < g.N) {
#pragma unroll
                    for (int r = 0; r < 16; ++r)
                        if (c0 + r < g.rows) out[(size_t)(c0 + r) * g.ld_part] = v[r] + w[r];
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_acc_empty[buf]);
            blk = seg_end;
            ++seg;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)g.tmem_cols) : "memory");
    }
    if (threadIdx.x == 0 && abort_flag) atomicExch(g.err, GEMM_ERR_TIMEOUT);
}

template <typename T>
__global__ void retile_kernel(const T* __restrict__ src, int rows, int K, int row_off, int k_blocks, long long total, int G,
                              bf16* __restrict__ dst) {
    const int chunks = K / 8;                                  // 8 consecutive inputs never straddle a 64-wide block
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < (size_t)rows * chunks; i += (size_t)gridDim.x * blockDim.x) {
        const int r = (int)(i / chunks), k0 = (int)(i % chunks) * 8;
        const int n = row_off + r;
        const long long slot = gemm_block_slot((long long)(n >> 7) * k_blocks + (k0 >> 6), total, G);
        bf16* out = dst + gemm_block_elem(slot, n & 127, k0 & 63);
        const T* in = src + (size_t)r * K + k0;
#pragma unroll
        for (int e = 0; e < 8; ++e) out[e] = (bf16)in[e];
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

}  // namespace

// A bf16 matrix [rows][K] (K contiguous) seen through boxes of 64 x box_rows elements, 128-byte swizzle.
anpd_status make_tmap_bf16(CUtensorMap* out, const void* base, int rows, int K, int box_rows, bool streamed) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return ANPD_ERR_CUDA;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)TILE_K, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          streamed ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        if (std::getenv("ANPD_VERBOSE")) std::fprintf(stderr, "[anpd] cuTensorMapEncodeTiled failed: %d (rows %d K %d box %d)\n", (int)r, rows, K, box_rows);
        return ANPD_ERR_CUDA;
    }
    return ANPD_OK;
}

size_t gemm_tiled_elems(const GemmPlan& p) { return (size_t)p.max_count * p.grid * TILE_M * TILE_K; }

anpd_status gemm_retile_enqueue(const GemmPlan& p, const void* src, bool src_is_f32, int rows, int row_off, bf16* dst_tiled, cudaStream_t st) {
    const size_t work = (size_t)rows * (p.K / 8);
    const int blocks = (int)std::min<size_t>((work + 255) / 256, 148 * 16);
    const long long total = (long long)p.m_tiles * p.k_blocks;
    if (src_is_f32) retile_kernel<float><<<blocks, 256, 0, st>>>((const float*)src, rows, p.K, row_off, p.k_blocks, total, p.grid, dst_tiled);
    else retile_kernel<bf16><<<blocks, 256, 0, st>>>((const bf16*)src, rows, p.K, row_off, p.k_blocks, total, p.grid, dst_tiled);
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}

// Cuts the (m_tile, k_block) grid of an [N][K] weight matrix into `grid` equal contiguous ranges and
// records, per tile, which CTA starts it and how many ranges (= partial sums) cover it.
void gemm_make_plan(GemmPlan* p, int N, int K, int num_sms) {
    p->N = N; p->K = K;
    p->m_tiles = (N + TILE_M - 1) / TILE_M;
    p->k_blocks = (K + TILE_K - 1) / TILE_K;
    const long long total = (long long)p->m_tiles * p->k_blocks;
    p->grid = (int)std::min<long long>(num_sms, total);
    p->max_count = (int)((total + p->grid - 1) / p->grid);
    p->first_cta.assign(p->m_tiles, 0);
    p->seg_count.assign(p->m_tiles, 0);
    p->max_segs = 0;
    for (int c = 0; c < p->grid; ++c) {
        const long long lo = (long long)c * total / p->grid, hi = (long long)(c + 1) * total / p->grid;
        for (long long t = lo / p->k_blocks; t * p->k_blocks < hi; ++t) {
            if (p->seg_count[t] == 0) p->first_cta[t] = c;
            p->seg_count[t] += 1;
        }
    }
    for (int t = 0; t < p->m_tiles; ++t) p->max_segs = std::max(p->max_segs, p->seg_count[t]);
    p->d_first_cta = nullptr;
    p->d_seg_count = nullptr;
}

int gemm_smem_bytes(int NB, int* stages_out) {
    const int stage_bytes = A_BYTES + 2 * NB * 128;
    // Five 16 KB weight blocks in flight per SM stream fastest on this part (measured: 10 in flight cost 5 % of the
    // step, 8 cost 3 %, 4 cost 2 %); wide activation tiles (prefill) leave room for fewer.
    int stages = std::min(RING_STAGES, (200 * 1024) / stage_bytes);
    if (stages_out) *stages_out = stages;
    return stages * stage_bytes + 1024;
}

anpd_status gemm_tc_enqueue(const GemmPlan& plan, const bf16* w_blocks, const CUtensorMap& map_hi, const CUtensorMap& map_lo,
                            int rows, int NB, float* part, size_t seg_stride, int ld_part, int* err, cudaStream_t st,
                            Profiler* prof) {
    static bool attr_set[64] = {false};
    if (first_call_on_device(attr_set)) {
        CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
    }
    GemmArgs g;
    g.part = part; g.seg_stride = seg_stride; g.ld_part = ld_part;
    g.N = plan.N; g.rows = rows; g.NB = NB;
    g.m_tiles = plan.m_tiles; g.k_blocks = plan.k_blocks;
    const int smem = gemm_smem_bytes(NB, &g.stages);
    int cols = 32;
    while (cols < 4 * NB) cols <<= 1;
    g.tmem_cols = cols;
    g.first_cta = plan.d_first_cta;
    g.err = err;
    LAUNCH(prof, st, KC_GEMM, 2.0 * (double)plan.N * (double)plan.K,
           (launch_k(gemm_tc_kernel, plan.grid, GEMM_THREADS, smem, st, w_blocks, map_hi, map_lo, g)));
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}
