// The forward of one decode step (paper Section 3.1, "Verification": one forward over the K+1 tokens of a step against
// the KV cache) as ONE persistent kernel, one CTA per SM.
//
// The step is bound by reading every weight once, so the design goal is that the weight stream never stops.  Every CTA
// walks the same program - per layer: QKV projection, attention, O projection, gate/up projection, down projection;
// then the LM head - and its share of each projection is a fixed range of 16 KB weight blocks (the same ranges and the
// same block storage as the stand-alone GEMM kernel, see gemm_block_slot).  Inside a CTA four roles run decoupled:
//
//   weight producer (1 thread)   walks the whole step's list of weight blocks and attention pages and keeps a deep
//                                shared-memory ring full; it depends on nothing but free ring slots (only a KV page that
//                                holds this step's own rows waits for those rows), so HBM keeps streaming while the
//                                other roles hand results from one projection to the next;
//   activation producer (1 warp) waits until the input tiles of a projection exist (per-tile flags in global memory
//                                written by the CTA that finished the tile), then brings them in by TMA;
//   MMA issuer (1 thread)        tcgen05.mma with the weight block as the 128-row operand and the step's rows (hi terms,
//                                then lo terms) as the N operand, accumulators in tensor memory, two in flight;
//   epilogue group (4 warps)     drains accumulators to per-segment partial sums; the CTA whose partial sum completes a
//                                128-feature tile (an arrival counter per tile) adds the tile's partial sums in segment
//                                order and does the elementwise work that follows the projection - rotary embedding and
//                                KV append, residual add, SwiGLU, vocabulary argmax - then raises the tile's flag.
//
// RMSNorm is deferred: the residual stream's producer writes x * gain (as hi + lo bf16 terms) and the tile's sum of
// squares; the consumer of the following projection multiplies its output features by 1 / rms(x), which commutes with
// the matrix product.  Attention items (one 128-key page of one kv head for one group of 8 rows) flow through the same
// ring: K page, then V^T page; the epilogue group does the softmax across tensor-memory lanes; the CTA that finishes a
// head's last page merges the pages in page order.
//
// Every sum has a fixed order that depends on shapes and absolute positions only (segments in order, pages in order,
// tiles in order), so a row's value does not depend on which other rows share the step: a greedy step and a
// draft-and-verify step give the same bits for the same position.  Every wait (mbarrier or flag) is bounded; a wait
// that gives up sets the error word the host reads after the step, and all other waits then end quickly.
#include "internal.h"
#include "tc_ptx.cuh"

#include <math_constants.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <vector>

typedef __nv_bfloat16 bf16;

namespace {

using namespace tc;

constexpr int ST_THREADS = 224;          // warp 0 weight producer, 1 MMA issuer, 2 activation producer, 3-6 epilogue group
constexpr int ST_MAX_STAGES = 12;
constexpr int W_BYTES = 16384;           // one weight block: 128 rows x 64 bf16, swizzled image
constexpr int SB = 2;                    // weight blocks per ring stage: a thread manages about one mbarrier operation per 90 cycles,
                                         // so a stage must carry enough bytes for the hand-over not to bound the stream
constexpr int QP_BYTES = 4096;           // attention Q operand / P operand: 16 rows (8 hi, 8 lo) x 128 columns
constexpr int SCRATCH_MIN = 8192;        // page maxima and sums while pages are merged: 2 x 8 rows x 128 pages
constexpr int ST_MAX_PAGES = 128;
constexpr int ST_ERR_TIMEOUT = 204;
constexpr int AQ = 8, AN = 16;           // query vectors per attention item, and the MMA's N (hi + lo terms)
constexpr unsigned FLAG_LIMIT = 1u << 21;
constexpr int TILE = 128;
constexpr int MAX_SEGS = 8;            // most partial sums a tile may have on this path

__device__ __forceinline__ int ld_acquire(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// arrival counter: one read-modify-write that publishes this thread's earlier writes and orders its later reads
__device__ __forceinline__ int atom_add_acq_rel(int* p, int v) {
    int old;
    asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}
__device__ __forceinline__ void red_add_release(int* p, int v) { asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory"); }
__device__ __forceinline__ void fence_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void group_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

__device__ __forceinline__ void split_bf16(float v, bf16& hi, bf16& lo) {
    hi = __float2bfloat16_rn(v);
    lo = __float2bfloat16_rn(v - __bfloat162float(hi));
}

__device__ __forceinline__ void tc_ld8(uint32_t taddr, float* v) {
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]) : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}

struct Ring {
    int s;
    uint32_t ph;
    int n;
    __device__ __forceinline__ void adv() { if (++s == n) { s = 0; ph ^= 1u; } }
};

// Byte offset of element (row n, column k) of a [16 rows][128 columns] bf16 operand held as two 64-column tiles in the
// 128-byte-swizzled K-major layout.
__device__ __forceinline__ int qp_offset(int n, int k) {
    const int kk = k & 63;
    return (k >> 6) * (AN * 128) + (n >> 3) * 1024 + (n & 7) * 128 + ((((kk >> 3) ^ (n & 7))) << 4) + (kk & 7) * 2;
}

// Activations of a projection are kept as the operand image the MMA reads, one k-block (64 inputs) after the other: per
// k-block nr rows of 128 bytes (rows 0 .. nr/2-1 the hi terms of the step's rows, then the lo terms) in the 128-byte-swizzled
// K-major layout, so that a k-block arrives with one linear copy.  Byte offset of element (operand row n, input k):
__device__ __forceinline__ size_t img_offset(int nr, int n, int k) {
    const int kk = k & 63;
    return (size_t)(k >> 6) * nr * 128 + (size_t)(n >> 3) * 1024 + (size_t)(n & 7) * 128 + (size_t)((((kk >> 3) ^ (n & 7))) << 4) + (size_t)(kk & 7) * 2;
}

struct AItem { int page, kvh, rg, pos_lo, pos_hi, seq; };

__global__ void __launch_bounds__(ST_THREADS, 1) step_kernel(const __grid_constant__ StepParams p, const int chunks, const int want_logits) {
    extern __shared__ __align__(1024) unsigned char st_smem_raw[];
    __shared__ uint64_t full[ST_MAX_STAGES], empty[ST_MAX_STAGES];
    __shared__ uint64_t acc_full[2], acc_empty[2], q_staged, s_full, p_staged, o_full;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag, s_last;
    __shared__ float s_rstd[64];
    __shared__ float s_red[4][64];
    __shared__ int s_redi[4][64];
    __shared__ float red_max[4][AQ], red_sum[2][4][AQ];

    pdl_trigger();
    const int S = p.stages, NR = 2 * p.rows, A_BYTES = NR * 128;     // NR: operand rows of the activations (hi terms, then lo terms)
    unsigned char* smem = st_smem_raw + ((1024u - (smem_u32(st_smem_raw) & 1023u)) & 1023u);
    unsigned char* ring_w = smem;
    unsigned char* ring_a = ring_w + (size_t)S * SB * W_BYTES;
    unsigned char* qbuf = ring_a + (size_t)S * SB * A_BYTES;
    unsigned char* pbuf = qbuf + QP_BYTES;
    float* scratch = (float*)(pbuf + QP_BYTES);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cta = blockIdx.x, G = gridDim.x;
    const int RG = p.rows / ANPD_ROWS;                 // groups of 8 rows (sequences)
    const int d_tiles = p.d / TILE, f_tiles = p.F / TILE;
    int tmem_cols = 32;
    while (tmem_cols < 2 * NR + 2 * AN) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < S; ++s) { mbar_init(&full[s], 2); mbar_init(&empty[s], 1); }     // full: weight producer + activation producer
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 4); }
        mbar_init(&q_staged, 1); mbar_init(&s_full, 1); mbar_init(&p_staged, 1); mbar_init(&o_full, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"((uint32_t)tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *((volatile uint32_t*)&tmem_slot);
    const uint32_t tmem_attn = tmem_base + (uint32_t)(2 * NR);
    volatile int* abortp = &abort_flag;

    pdl_wait();                                        // the row plan and the cleared flags come from earlier nodes of the step

    // ---- bounded waits: on giving up they raise the CTA's abort flag and the step's error word ----
    auto mwait = [&](uint64_t* bar, uint32_t parity) -> bool {
        if (mbar_wait(bar, parity, abortp)) return true;
        atomicExch(p.err, ST_ERR_TIMEOUT);
        return false;
    };
    auto fwait = [&](const int* f, int need) -> bool {    // until the counter at f has reached `need`
        for (unsigned i = 0; i < FLAG_LIMIT; ++i) {
            if (ld_acquire(f) >= need) return true;
            __nanosleep(40);
            if ((i & 63u) == 63u) {
                if (*abortp) return false;
                if (ld_acquire(p.err) != 0) { *abortp = 1; return false; }
            }
        }
        *abortp = 1;
        atomicExch(p.err, ST_ERR_TIMEOUT);
        return false;
    };
    auto gemm_range = [&](const StepGemm& g, long long& lo, long long& hi) {
        if (cta >= g.grid) { lo = 0; hi = 0; return; }
        const long long total = (long long)g.m_tiles * g.k_blocks;
        lo = (long long)cta * total / g.grid;
        hi = (long long)(cta + 1) * total / g.grid;
    };
    const int n_items = chunks * p.Hkv * RG;
    auto item_at = [&](int it, AItem& a) -> bool {      // false: the page lies beyond everything the group's rows may see
        const int per_page = p.Hkv * RG;
        a.page = it / per_page;
        const int rem = it - a.page * per_page;
        a.kvh = rem / RG; a.rg = rem - a.kvh * RG;
        a.pos_lo = p.row_pos[a.rg * ANPD_ROWS];
        a.pos_hi = p.row_pos[a.rg * ANPD_ROWS + ANPD_ROWS - 1];
        a.seq = p.row_seq[a.rg * ANPD_ROWS];
        return a.page * KV_PAGE <= a.pos_hi;
    };
    auto sync_at = [&](int layer, int off) -> int* { return p.sync + (size_t)layer * p.sync_stride + off; };
    // optional time stamps of one CTA (a debugging aid): slot k of projection g (0 QKV, 1 O, 2 gate/up, 3 down) of layer l
    auto stamp_gemm = [&](int l, int g, int k) {
        if (p.trace && cta == p.trace_cta && l < p.L) {
            unsigned long long t;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
            p.trace[5 * p.L + 2 + (l * 4 + g) * 3 + k] = t;
        }
    };

    if (warp == 0) {
        // =====================================================================================================
        // weight / page producer
        // =====================================================================================================
        if (lane == 0) {
            const uint64_t pol_w = policy_evict_first();
            Ring c{0, 0u, S};
            bool ok = true;
            auto prod_gemm = [&](const StepGemm& g, const bf16* w) -> bool {
                long long lo, hi;
                gemm_range(g, lo, hi);
                for (long long i = 0; i < hi - lo; i += SB) {
                    const int n = (int)min((long long)SB, hi - lo - i);
                    if (!mwait(&empty[c.s], c.ph ^ 1u)) return false;
                    mbar_expect_tx(&full[c.s], (uint32_t)(n * W_BYTES));
                    for (int b = 0; b < n; ++b)
                        bulk_load(ring_w + (size_t)(c.s * SB + b) * W_BYTES, w + (size_t)((i + b) * g.grid + cta) * (TILE * 64), W_BYTES, &full[c.s], pol_w);
                    c.adv();
                }
                return true;
            };
            auto prod_attn = [&](int l) -> bool {
                for (int it = cta; it < n_items; it += G) {
                    AItem a;
                    if (!item_at(it, a)) continue;
                    if (a.page * KV_PAGE + KV_PAGE - 1 >= a.pos_lo) {
                        // the page holds rows this step appends: wait until the QKV projection's tiles are all finished
                        if (!fwait(sync_at(l, p.o_dqkv), p.g[GK_QKV].m_tiles)) return false;
                        fence_async_global();
                    }
                    const int row = l * p.layer_rows + (p.page_table[a.seq * p.pages_per_seq + a.page] * p.Hkv + a.kvh) * KV_PAGE;
                    for (int q = 0; q < 2; ++q) {              // one stage for the K page, one for the V^T page
                        if (!mwait(&empty[c.s], c.ph ^ 1u)) return false;
                        mbar_expect_tx(&full[c.s], 2 * W_BYTES);
                        tma_load_2d(ring_w + (size_t)(c.s * SB) * W_BYTES, q == 0 ? &p.map_k : &p.map_v, 0, row, &full[c.s], pol_w);
                        tma_load_2d(ring_w + (size_t)(c.s * SB + 1) * W_BYTES, q == 0 ? &p.map_k : &p.map_v, 64, row, &full[c.s], pol_w);
                        c.adv();
                    }
                }
                return true;
            };
            for (int l = 0; l < p.L && ok; ++l) {
                const StepLayer lay = p.layers[l];
                ok = prod_gemm(p.g[GK_QKV], lay.wqkv) && prod_attn(l) && prod_gemm(p.g[GK_O], lay.wo) && prod_gemm(p.g[GK_GU], lay.wgu) &&
                     prod_gemm(p.g[GK_DOWN], lay.wd);
            }
            ok = ok && prod_gemm(p.g[GK_LM], p.lm_head);
            if (!ok) {
                // gave up: the copies already requested must land before the CTA may exit; they need no more than microseconds
                const long long t0 = clock64();
                while (clock64() - t0 < (1ll << 21)) {}
            }
        }
    } else if (warp == 2) {
        // =====================================================================================================
        // activation producer
        // =====================================================================================================
        const uint64_t pol_a = policy_evict_last();
        Ring c{0, 0u, S};
        bool ok = true;
        // `done` counts the finished tiles of the phase that writes this projection's input; `need` is all of them
        auto act_gemm = [&](const StepGemm& g, const unsigned char* img, const int* done, int need, int tl_, int tg_) -> bool {
            long long lo, hi;
            gemm_range(g, lo, hi);
            int res = 1;
            if (lane == 0) {
                if (hi > lo && !fwait(done, need)) res = 0;
                stamp_gemm(tl_, tg_, 0);
                fence_async_global();
                int kb = (hi > lo) ? (int)(lo % g.k_blocks) : 0;
                for (long long i = 0; i < hi - lo && res; i += SB) {
                    const int n = (int)min((long long)SB, hi - lo - i);
                    if (!mwait(&empty[c.s], c.ph ^ 1u)) { res = 0; break; }
                    unsigned char* sa = ring_a + (size_t)(c.s * SB) * A_BYTES;
                    mbar_expect_tx(&full[c.s], (uint32_t)(n * A_BYTES));
                    if (kb + n <= g.k_blocks) {             // consecutive k-blocks are consecutive in the image: one copy
                        bulk_load(sa, img + (size_t)kb * A_BYTES, (uint32_t)(n * A_BYTES), &full[c.s], pol_a);
                        kb += n;
                        if (kb == g.k_blocks) kb = 0;
                    } else {
                        for (int b = 0; b < n; ++b) {
                            bulk_load(sa + (size_t)b * A_BYTES, img + (size_t)kb * A_BYTES, (uint32_t)A_BYTES, &full[c.s], pol_a);
                            if (++kb == g.k_blocks) kb = 0;
                        }
                    }
                    c.adv();
                }
            }
            res = __shfl_sync(0xffffffffu, res, 0);
            c.s = __shfl_sync(0xffffffffu, c.s, 0);
            c.ph = __shfl_sync(0xffffffffu, c.ph, 0);
            return res != 0;
        };
        auto act_attn = [&]() -> bool {
            int res = 1;
            if (lane == 0) {
                for (int it = cta; it < n_items && res; it += G) {
                    AItem a;
                    if (!item_at(it, a)) continue;
                    for (int q = 0; q < 2; ++q) {
                        if (!mwait(&empty[c.s], c.ph ^ 1u)) { res = 0; break; }
                        mbar_arrive(&full[c.s]);            // a page stage carries no activation tile: this role's arrival only
                        c.adv();
                    }
                }
            }
            res = __shfl_sync(0xffffffffu, res, 0);
            c.s = __shfl_sync(0xffffffffu, c.s, 0);
            c.ph = __shfl_sync(0xffffffffu, c.ph, 0);
            return res != 0;
        };
        for (int l = 0; l < p.L && ok; ++l) {
            ok = act_gemm(p.g[GK_QKV], p.imgA, sync_at(l, p.o_dh), d_tiles, l, 0) && act_attn() &&
                 act_gemm(p.g[GK_O], p.img_ao, sync_at(l, p.o_dao), p.rows * p.Hq, l, 1) && act_gemm(p.g[GK_GU], p.imgB, sync_at(l, p.o_dhB), d_tiles, l, 2) &&
                 act_gemm(p.g[GK_DOWN], p.img_act, sync_at(l, p.o_dact), f_tiles, l, 3);
        }
        ok = ok && act_gemm(p.g[GK_LM], p.imgA, sync_at(p.L, p.o_dh), d_tiles, p.L, 0);
        if (!ok && lane == 0) {
            const long long t0 = clock64();
            while (clock64() - t0 < (1ll << 21)) {}
        }
    } else if (warp == 1) {
        // =====================================================================================================
        // MMA issuer
        // =====================================================================================================
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NR >> 3) << 17) | ((uint32_t)(TILE >> 4) << 24);
            const uint32_t idesc_attn = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(AN >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
            Ring c{0, 0u, S};
            int seg = 0;
            uint32_t aj = 0;                            // attention items issued so far (parity of the item barriers)
            bool ok = true;
            auto mma_gemm = [&](const StepGemm& g, int tl_, int tg_) -> bool {
                long long lo, hi;
                gemm_range(g, lo, hi);
                long long blk = lo;
                bool first = true;
                long long w_f = 0, w_acc = 0;
                const bool tr = p.trace && cta == p.trace_cta;
                while (blk < hi) {
                    const int tile = (int)(blk / g.k_blocks);
                    const long long seg_end = min(hi, (long long)(tile + 1) * g.k_blocks);
                    const int buf = seg & 1;
                    long long t0 = tr ? clock64() : 0;
                    if (!mwait(&acc_empty[buf], (uint32_t)(((seg >> 1) & 1) ^ 1))) return false;
                    if (tr) w_acc += clock64() - t0;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + (uint32_t)(buf * NR);
                    uint32_t acc = 0;
                    for (; blk < seg_end; ++blk) {
                        const int b = (int)((blk - lo) % SB);       // position of the block in its stage
                        if (b == 0) {
                            t0 = tr ? clock64() : 0;
                            if (!mwait(&full[c.s], c.ph)) return false;
                            if (tr) w_f += clock64() - t0;
                            if (first) { stamp_gemm(tl_, tg_, 1); first = false; }
                            tc_fence_after();
                        }
                        const uint64_t da = make_smem_desc(smem_u32(ring_w + (size_t)(c.s * SB + b) * W_BYTES));
                        const uint64_t db = make_smem_desc(smem_u32(ring_a + (size_t)(c.s * SB + b) * A_BYTES));
#pragma unroll
                        for (int k16 = 0; k16 < 4; ++k16) {
                            const uint64_t adv = (uint64_t)(k16 * 2);
                            tc_mma_bf16(d_tmem, da + adv, db + adv, idesc, acc);
                            acc = 1;
                        }
                        if (b == SB - 1 || blk + 1 == hi) {          // the stage's last block
                            tc_commit(&empty[c.s]);
                            c.adv();
                        }
                    }
                    tc_commit(&acc_full[buf]);
                    ++seg;
                }
                stamp_gemm(tl_, tg_, 2);
                if (tr && tl_ < p.L) {
                    unsigned long long* q = p.trace + 17 * p.L + 2 + (tl_ * 4 + tg_) * 3;
                    q[0] = (unsigned long long)w_f; q[1] = 0; q[2] = (unsigned long long)w_acc;
                }
                return true;
            };
            auto mma_attn = [&]() -> bool {
                for (int it = cta; it < n_items; it += G) {
                    AItem a;
                    if (!item_at(it, a)) continue;
                    const uint32_t par = aj & 1u;
                    const uint32_t d_tmem = tmem_attn + par * AN;
                    if (!mwait(&full[c.s], c.ph) || !mwait(&q_staged, par)) return false;
                    tc_fence_after();
#pragma unroll
                    for (int k16 = 0; k16 < 8; ++k16) {
                        const uint64_t adv = (uint64_t)((k16 & 3) * 2);
                        tc_mma_bf16(d_tmem, make_smem_desc(smem_u32(ring_w + (size_t)(c.s * SB + (k16 >> 2)) * W_BYTES)) + adv,
                                    make_smem_desc(smem_u32(qbuf + (k16 >> 2) * (AN * 128))) + adv, idesc_attn, k16 > 0 ? 1u : 0u);
                    }
                    tc_commit(&s_full);
                    tc_commit(&empty[c.s]);
                    c.adv();
                    if (!mwait(&full[c.s], c.ph) || !mwait(&p_staged, par)) return false;
                    tc_fence_after();
#pragma unroll
                    for (int k16 = 0; k16 < 8; ++k16) {
                        const uint64_t adv = (uint64_t)((k16 & 3) * 2);
                        tc_mma_bf16(d_tmem, make_smem_desc(smem_u32(ring_w + (size_t)(c.s * SB + (k16 >> 2)) * W_BYTES)) + adv,
                                    make_smem_desc(smem_u32(pbuf + (k16 >> 2) * (AN * 128))) + adv, idesc_attn, k16 > 0 ? 1u : 0u);
                    }
                    tc_commit(&o_full);
                    tc_commit(&empty[c.s]);
                    c.adv();
                    ++aj;
                }
                return true;
            };
            for (int l = 0; l < p.L && ok; ++l)
                ok = mma_gemm(p.g[GK_QKV], l, 0) && mma_attn() && mma_gemm(p.g[GK_O], l, 1) && mma_gemm(p.g[GK_GU], l, 2) && mma_gemm(p.g[GK_DOWN], l, 3);
            ok = ok && mma_gemm(p.g[GK_LM], p.L, 0);
        }
    } else {
        // =====================================================================================================
        // epilogue group: 128 threads; e indexes features / keys / dimensions, quad is the warp's tensor-memory lane quarter
        // =====================================================================================================
        const int quad = warp & 3;
        const int tl = quad * 32 + lane;                 // the tensor-memory lane this thread may read
        const int e = (warp - 3) * 32 + lane;            // 0..127
        const int ew = warp - 3;
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        int seg = 0;
        uint32_t aj = 0;
        bool ok = true;
        const int rows = p.rows;
        const float inv_d = 1.0f / (float)p.d;

        // One thread polls the barrier (a short sleep between polls); the other 127 wait at the hardware barrier, where they
        // cost neither issue slots nor shared-memory bandwidth.
        auto gwait = [&](uint64_t* bar, uint32_t parity) -> bool {
            if (e == 0) {
                bool got = false;
                for (unsigned i = 0; i < WAIT_LIMIT && !got; ++i) {
                    got = mbar_try_wait(bar, parity);
                    if (!got) {
                        __nanosleep(32);
                        if ((i & 255u) == 255u && *abortp) break;
                    }
                }
                if (!got) { *abortp = 1; atomicExch(p.err, ST_ERR_TIMEOUT); }
            }
            group_bar();
            return *abortp == 0;
        };
        // 1 / rms of every row from the tile sums of squares: all threads fetch, then one thread per row adds in tile order
        auto compute_rstd = [&](const float* ss) {
            const int n = d_tiles * rows;
            for (int i = e; i < n; i += 128) scratch[i] = __ldcg(ss + i);
            group_bar();
            if (e < rows) {
                float acc = 0.0f;
                for (int t = 0; t < d_tiles; ++t) acc += scratch[t * rows + e];
                s_rstd[e] = rsqrtf(acc * inv_d + p.eps);
            }
            group_bar();
        };
        // sums of the partial sums of 8 consecutive rows of one feature, segments in order; every load is issued
        // before the first is used
        auto sum8 = [&](const float* base, int ld, unsigned long long seg_stride, int nseg, float* out) {
            float v[8][MAX_SEGS];
#pragma unroll
            for (int r = 0; r < 8; ++r)
#pragma unroll
                for (int sg = 0; sg < MAX_SEGS; ++sg)
                    v[r][sg] = (sg < nseg) ? __ldcg(base + (size_t)r * ld + (size_t)sg * seg_stride) : 0.0f;
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                float a = 0.0f;
#pragma unroll
                for (int sg = 0; sg < MAX_SEGS; ++sg)
                    if (sg < nseg) a += v[r][sg];
                out[r] = a;
            }
        };
        // after a tail's stores: make them visible (to plain loads and to TMA reads of other CTAs), then count the tile as done
        auto publish = [&](int* done) {
            fence_async_global();
            group_bar();
            if (e == 0) red_add_release(done, 1);
        };
        // x (+)= v per row for one 128-column tile; h = x * gain as hi + lo; the tile's sum of squares per row
        auto resid_tail = [&](int tile, const StepGemm* g, const float* gain, unsigned char* img, float* ss) {
            const int n = tile * TILE + e;
            const float gn = gain[n];
            const int nseg = g ? g->seg_count[tile] : 0;
            for (int r0 = 0; r0 < rows; r0 += 8) {
                float xn[8];
                if (g) {
                    float xo[8], v[8];
#pragma unroll
                    for (int r = 0; r < 8; ++r) xo[r] = __ldcg(p.x + (size_t)(r0 + r) * p.d + n);
                    sum8(g->part + (size_t)r0 * g->ld_part + n, g->ld_part, g->seg_stride, nseg, v);
#pragma unroll
                    for (int r = 0; r < 8; ++r) xn[r] = xo[r] + v[r];
                } else {
                    int tok[8];
#pragma unroll
                    for (int r = 0; r < 8; ++r) tok[r] = p.row_tok[r0 + r];
#pragma unroll
                    for (int r = 0; r < 8; ++r) xn[r] = __bfloat162float(p.embed[(size_t)tok[r] * p.d + n]);
                }
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    p.x[(size_t)(r0 + r) * p.d + n] = xn[r];
                    bf16 hi, lo;
                    split_bf16(xn[r] * gn, hi, lo);
                    *(bf16*)(img + img_offset(NR, r0 + r, n)) = hi;
                    *(bf16*)(img + img_offset(NR, rows + r0 + r, n)) = lo;
                }
                float sq[8];
#pragma unroll
                for (int r = 0; r < 8; ++r) sq[r] = xn[r] * xn[r];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                    for (int r = 0; r < 8; ++r) sq[r] += __shfl_xor_sync(0xffffffffu, sq[r], o);
                if (lane == 0)
#pragma unroll
                    for (int r = 0; r < 8; ++r) s_red[ew][r0 + r] = sq[r];
            }
            group_bar();
            if (e < rows) ss[(size_t)tile * rows + e] = ((s_red[0][e] + s_red[1][e]) + s_red[2][e]) + s_red[3][e];
        };
        auto qkv_tail = [&](int l, int tile) {
            const StepGemm& g = p.g[GK_QKV];
            const int half = p.hd >> 1;
            const int pr_i = e & 63, rh = e >> 6;
            const int head_in_tile = pr_i / half, i = pr_i - head_in_tile * half;
            const int na = tile * TILE + head_in_tile * p.hd + i, nb = na + half;
            const int head = na / p.hd;
            const int nseg = g.seg_count[tile];
            bf16* kp = p.kpool + (size_t)l * p.layer_elems;
            bf16* vp = p.vpool + (size_t)l * p.layer_elems;
            // thread (feature pair, half of the rows): rows 4 * rh .. + 3 of every group of 8
            for (int r0 = 4 * rh; r0 < rows; r0 += 8) {
                float va[4][MAX_SEGS], vb[4][MAX_SEGS], cs[4], sn[4];
                int pos[4];
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    pos[r] = p.row_pos[r0 + r];
                    const float* pa = g.part + (size_t)(r0 + r) * g.ld_part;
#pragma unroll
                    for (int sg = 0; sg < MAX_SEGS; ++sg) {
                        va[r][sg] = (sg < nseg) ? __ldcg(pa + (size_t)sg * g.seg_stride + na) : 0.0f;
                        vb[r][sg] = (sg < nseg) ? __ldcg(pa + (size_t)sg * g.seg_stride + nb) : 0.0f;
                    }
                }
#pragma unroll
                for (int r = 0; r < 4; ++r) { cs[r] = p.rope_cos[(size_t)pos[r] * half + i]; sn[r] = p.rope_sin[(size_t)pos[r] * half + i]; }
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const int row = r0 + r;
                    float a = 0.0f, b = 0.0f;
#pragma unroll
                    for (int sg = 0; sg < MAX_SEGS; ++sg)
                        if (sg < nseg) { a += va[r][sg]; b += vb[r][sg]; }
                    a *= s_rstd[row]; b *= s_rstd[row];
                    if (head < p.Hq + p.Hkv) {
                        const float ra = a * cs[r] - b * sn[r], rb = b * cs[r] + a * sn[r];
                        a = ra; b = rb;
                    }
                    if (head < p.Hq) {
                        const size_t o = (size_t)row * p.dq + (size_t)head * p.hd + i;
                        split_bf16(a * p.q_scale, p.q_hi[o], p.q_lo[o]);
                        split_bf16(b * p.q_scale, p.q_hi[o + half], p.q_lo[o + half]);
                    } else if (p.row_ok[row]) {
                        const bool is_k = head < p.Hq + p.Hkv;
                        const int kvh = is_k ? head - p.Hq : head - p.Hq - p.Hkv;
                        const int page = p.page_table[p.row_seq[row] * p.pages_per_seq + pos[r] / KV_PAGE];
                        bf16* pg = (is_k ? kp : vp) + ((size_t)page * p.Hkv + kvh) * KV_PAGE * p.hd;
                        if (is_k) {
                            pg[(size_t)(pos[r] % KV_PAGE) * p.hd + i] = __float2bfloat16_rn(a);
                            pg[(size_t)(pos[r] % KV_PAGE) * p.hd + i + half] = __float2bfloat16_rn(b);
                        } else {
                            pg[(size_t)i * KV_PAGE + (pos[r] % KV_PAGE)] = __float2bfloat16_rn(a);
                            pg[(size_t)(i + half) * KV_PAGE + (pos[r] % KV_PAGE)] = __float2bfloat16_rn(b);
                        }
                    }
                }
            }
        };
        auto gu_tail = [&](int jt) {
            const StepGemm& g = p.g[GK_GU];
            const int j = jt * TILE + e;
            const int ng = g.seg_count[jt], nu = g.seg_count[jt + f_tiles];
            const int nmax = max(ng, nu);
            for (int r0 = 0; r0 < rows; r0 += 8) {
                float gte[8], up[8];
#pragma unroll
                for (int r = 0; r < 8; ++r) { gte[r] = 0.0f; up[r] = 0.0f; }
                const float* pg = g.part + (size_t)r0 * g.ld_part + j;
                // gate and up partial sums are requested together, four segments at a time, and added in segment order
                for (int s0 = 0; s0 < nmax; s0 += 4) {
                    float vg[8][4], vu[8][4];
#pragma unroll
                    for (int r = 0; r < 8; ++r)
#pragma unroll
                        for (int sg = 0; sg < 4; ++sg) {
                            vg[r][sg] = (s0 + sg < ng) ? __ldcg(pg + (size_t)r * g.ld_part + (size_t)(s0 + sg) * g.seg_stride) : 0.0f;
                            vu[r][sg] = (s0 + sg < nu) ? __ldcg(pg + p.F + (size_t)r * g.ld_part + (size_t)(s0 + sg) * g.seg_stride) : 0.0f;
                        }
#pragma unroll
                    for (int r = 0; r < 8; ++r)
#pragma unroll
                        for (int sg = 0; sg < 4; ++sg) {
                            if (s0 + sg < ng) gte[r] += vg[r][sg];
                            if (s0 + sg < nu) up[r] += vu[r][sg];
                        }
                }
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    const float a = gte[r] * s_rstd[r0 + r], b = up[r] * s_rstd[r0 + r];
                    const float v = a / (1.0f + expf(-a)) * b;
                    bf16 hi, lo;
                    split_bf16(v, hi, lo);
                    *(bf16*)(p.img_act + img_offset(NR, r0 + r, j)) = hi;
                    *(bf16*)(p.img_act + img_offset(NR, rows + r0 + r, j)) = lo;
                }
            }
        };
        auto lm_tail = [&](int tile) {
            const StepGemm& g = p.g[GK_LM];
            const int n = tile * TILE + e;
            const int nseg = g.seg_count[tile];
            for (int r0 = 0; r0 < rows; r0 += 8) {
                float z[8];
                int idx[8];
                if (n < p.V) {
                    sum8(g.part + (size_t)r0 * g.ld_part + n, g.ld_part, g.seg_stride, nseg, z);
#pragma unroll
                    for (int r = 0; r < 8; ++r) {
                        z[r] *= s_rstd[r0 + r];
                        idx[r] = n;
                        if (want_logits) p.logits[(size_t)(r0 + r) * p.V + n] = z[r];
                    }
                } else {
#pragma unroll
                    for (int r = 0; r < 8; ++r) { z[r] = -CUDART_INF_F; idx[r] = 0x7fffffff; }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                    for (int r = 0; r < 8; ++r) {
                        const float oz = __shfl_xor_sync(0xffffffffu, z[r], o);
                        const int oi = __shfl_xor_sync(0xffffffffu, idx[r], o);
                        if (oz > z[r] || (oz == z[r] && oi < idx[r])) { z[r] = oz; idx[r] = oi; }
                    }
                if (lane == 0)
#pragma unroll
                    for (int r = 0; r < 8; ++r) { s_red[ew][r0 + r] = z[r]; s_redi[ew][r0 + r] = idx[r]; }
            }
            group_bar();
            if (e < rows) {
                float z = s_red[0][e];
                int idx = s_redi[0][e];
                for (int w = 1; w < 4; ++w)
                    if (s_red[w][e] > z || (s_red[w][e] == z && s_redi[w][e] < idx)) { z = s_red[w][e]; idx = s_redi[w][e]; }
                p.amax_val[(size_t)e * g.m_tiles + tile] = z;
                p.amax_idx[(size_t)e * g.m_tiles + tile] = idx;
            }
        };
        // merge the pages of one (row, query head): pages in ascending order, four interleaved running sums added in a fixed
        // order, as the stand-alone combine kernel keeps them.  Thread = output dimension.
        auto combine_unit = [&](int row, int hq) {
            const int nc = p.row_pos[row] / KV_PAGE + 1;
            const size_t base = ((size_t)row * p.Hq + hq) * p.pages_per_seq;
            float M = -CUDART_INF_F;
            for (int c0 = 0; c0 < nc; c0 += 8) {
                float mv[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) mv[k] = (c0 + k < nc) ? __ldcg(p.pm + base + c0 + k) : -CUDART_INF_F;
#pragma unroll
                for (int k = 0; k < 8; ++k) M = fmaxf(M, mv[k]);
            }
            float L = 0.0f;
            float o[4] = {0.f, 0.f, 0.f, 0.f};
            for (int c0 = 0; c0 < nc; c0 += 8) {
                float mv[8], lv[8], ov[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const bool in = c0 + k < nc;
                    mv[k] = in ? __ldcg(p.pm + base + c0 + k) : 0.0f;
                    lv[k] = in ? __ldcg(p.pl + base + c0 + k) : 0.0f;
                    ov[k] = in ? __ldcg(p.po + (base + c0 + k) * 128 + e) : 0.0f;
                }
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if (c0 + k < nc) {
                        const float w = exp2f(mv[k] - M);
                        L = fmaf(lv[k], w, L);
                        o[k & 3] = fmaf(ov[k], w, o[k & 3]);
                    }
            }
            const float t = ((o[0] + o[1]) + o[2]) + o[3];
            bf16 hi, lo;
            split_bf16(t / L, hi, lo);
            *(bf16*)(p.img_ao + img_offset(NR, row, hq * 128 + e)) = hi;
            *(bf16*)(p.img_ao + img_offset(NR, rows + row, hq * 128 + e)) = lo;
        };

        // kind: which tail follows the projection
        auto epi_gemm = [&](int kind, int l) -> bool {
            const StepGemm& g = p.g[kind];
            long long lo, hi;
            gemm_range(g, lo, hi);
            long long blk = lo;
            while (blk < hi) {
                const int tile = (int)(blk / g.k_blocks);
                const long long seg_end = min(hi, (long long)(tile + 1) * g.k_blocks);
                const int buf = seg & 1;
                if (!gwait(&acc_full[buf], (uint32_t)((seg >> 1) & 1))) return false;
                tc_fence_after();
                if (blk == lo && kind != GK_O && kind != GK_DOWN) {
                    // First accumulator of the phase: the MMAs that filled it read the phase's whole input, so the input's tile
                    // sums of squares are complete.  1 / rms of every row, once per phase, while the weights keep streaming.
                    compute_rstd(kind == GK_GU ? p.ssB : p.ssA);
                }
                const int ordinal = cta - g.first_cta[tile];
                const int n = tile * TILE + tl;
                float* out = g.part + (size_t)ordinal * g.seg_stride + n;
                if (rows == 8) {                            // hi terms in columns 0-7, lo terms in 8-15: one load
                    float v[16];
                    tc_ld16(tmem_base + lane_addr + (uint32_t)(buf * NR), v);
                    if (n < g.N) {
#pragma unroll
                        for (int r = 0; r < 8; ++r) out[(size_t)r * g.ld_part] = v[r] + v[8 + r];
                    }
                } else {
                    for (int c0 = 0; c0 < rows; c0 += 8) {
                        float v[8], w[8];
                        tc_ld8(tmem_base + lane_addr + (uint32_t)(buf * NR + c0), v);
                        tc_ld8(tmem_base + lane_addr + (uint32_t)(buf * NR + rows + c0), w);
                        if (n < g.N) {
#pragma unroll
                            for (int r = 0; r < 8; ++r) out[(size_t)(c0 + r) * g.ld_part] = v[r] + w[r];
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc_empty[buf]);
                blk = seg_end;
                ++seg;
                // arrival: the CTA that completes the tile (or the gate/up pair of tiles) runs the tail
                group_bar();
                if (e == 0) {
                    int* cnt;
                    int target;
                    if (kind == GK_QKV) { cnt = sync_at(l, p.o_cqkv) + tile; target = g.seg_count[tile]; }
                    else if (kind == GK_O) { cnt = sync_at(l, p.o_co) + tile; target = g.seg_count[tile]; }
                    else if (kind == GK_GU) { const int jt = tile % f_tiles; cnt = sync_at(l, p.o_cgu) + jt; target = g.seg_count[jt] + g.seg_count[jt + f_tiles]; }
                    else if (kind == GK_DOWN) { cnt = sync_at(l, p.o_cdown) + tile; target = g.seg_count[tile]; }
                    else { cnt = sync_at(l, p.o_clm) + tile; target = g.seg_count[tile]; }
                    const int old = atom_add_acq_rel(cnt, 1);
                    s_last = (old == target - 1) ? 1 : 0;
                }
                group_bar();
                if (s_last) {
                    if (kind == GK_QKV) { qkv_tail(l, tile); publish(sync_at(l, p.o_dqkv)); }
                    else if (kind == GK_O) { resid_tail(tile, &g, p.layers[l].ffn_norm, p.imgB, p.ssB); publish(sync_at(l, p.o_dhB)); }
                    else if (kind == GK_GU) { const int jt = tile % f_tiles; gu_tail(jt); publish(sync_at(l, p.o_dact)); }
                    else if (kind == GK_DOWN) {
                        resid_tail(tile, &g, (l + 1 < p.L) ? p.layers[l + 1].attn_norm : p.final_norm, p.imgA, p.ssA);
                        publish(sync_at(l + 1, p.o_dh));
                    } else { lm_tail(tile); }
                }
                group_bar();                               // s_last and the reduction scratch are free again
            }
            return true;
        };
        auto epi_attn = [&](int l) -> bool {
            // the queries (and this step's K/V rows) exist once every tile of the QKV projection is finished
            if (e == 0 && !fwait(sync_at(l, p.o_dqkv), p.g[GK_QKV].m_tiles)) *abortp = 1;
            group_bar();
            if (*abortp) return false;
            auto fetch_q = [&](const AItem& a, uint4* regs) {
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int idx = e + u * 128;            // 16 operand rows x 16 chunks of 16 bytes
                    const int n = idx >> 4, c16 = idx & 15;
                    const int r = n & 7;
                    const bf16* src = (n < AQ ? p.q_hi : p.q_lo) + (size_t)(a.rg * ANPD_ROWS + r) * p.dq + (size_t)a.kvh * 128 + c16 * 8;
                    regs[u] = __ldcg((const uint4*)src);
                }
            };
            auto stage_q = [&](const uint4* regs) {
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int idx = e + u * 128;
                    *(uint4*)(qbuf + qp_offset(idx >> 4, (idx & 15) * 8)) = regs[u];
                }
            };
            int it = cta;
            int n_mine = 0;
            AItem cur, nxt;
            while (it < n_items && !item_at(it, cur)) it += G;
            if (it < n_items) {
                uint4 qr[2];
                fetch_q(cur, qr);
                stage_q(qr);
                fence_async_smem();
                group_bar();
                if (e == 0) mbar_arrive(&q_staged);
            }
            while (it < n_items) {
                const uint32_t par = aj & 1u;
                int it_next = it + G;
                while (it_next < n_items && !item_at(it_next, nxt)) it_next += G;
                const bool more = it_next < n_items;
                if (!gwait(&s_full, par)) return false;
                tc_fence_after();
                uint4 qr[2];
                if (more) fetch_q(nxt, qr);
                float s[AQ];
                {
                    float v[AN];
                    tc_ld16(tmem_attn + par * AN + lane_addr, v);
#pragma unroll
                    for (int q = 0; q < AQ; ++q) s[q] = v[q] + v[AQ + q];
                }
                const int key = cur.page * KV_PAGE + tl;
#pragma unroll
                for (int q = 0; q < AQ; ++q) {
                    if (key > cur.pos_lo + q) s[q] = -CUDART_INF_F;
                    float mx = s[q];
                    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                    if (lane == 0) red_max[quad][q] = mx;
                }
                tc_fence_before();
                group_bar();
                float m[AQ];
#pragma unroll
                for (int q = 0; q < AQ; ++q) {
                    m[q] = fmaxf(fmaxf(red_max[0][q], red_max[1][q]), fmaxf(red_max[2][q], red_max[3][q]));
                    const float pw = (m[q] == -CUDART_INF_F) ? 0.0f : exp2f(s[q] - m[q]);
                    const bf16 h = __float2bfloat16_rn(pw);
                    const bf16 lw = __float2bfloat16_rn(pw - __bfloat162float(h));
                    *(bf16*)(pbuf + qp_offset(q, tl)) = h;
                    *(bf16*)(pbuf + qp_offset(AQ + q, tl)) = lw;
                    float sum = pw;
                    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
                    if (lane == 0) red_sum[par][quad][q] = sum;
                }
                if (more) stage_q(qr);                      // the first product has finished reading the previous queries
                fence_async_smem();
                group_bar();
                if (e == 0) {
                    mbar_arrive(&p_staged);
                    if (more) mbar_arrive(&q_staged);
                }
                if (e < AQ) {
                    const size_t out = ((size_t)(cur.rg * ANPD_ROWS + e) * p.Hq + cur.kvh) * p.pages_per_seq + cur.page;
                    float mt = m[0];
#pragma unroll
                    for (int q = 1; q < AQ; ++q) mt = (q == e) ? m[q] : mt;
                    p.pm[out] = mt;
                    p.pl[out] = (red_sum[par][0][e] + red_sum[par][1][e]) + (red_sum[par][2][e] + red_sum[par][3][e]);
                }
                if (!gwait(&o_full, par)) return false;
                tc_fence_after();
                {
                    float v[AN];
                    tc_ld16(tmem_attn + par * AN + lane_addr, v);
#pragma unroll
                    for (int q = 0; q < AQ; ++q) {
                        const size_t out = ((size_t)(cur.rg * ANPD_ROWS + q) * p.Hq + cur.kvh) * p.pages_per_seq + cur.page;
                        p.po[out * 128 + tl] = v[q] + v[AQ + q];
                    }
                }
                tc_fence_before();
                ++n_mine;
                ++aj;
                cur = nxt;
                it = it_next;
            }
            // Every CTA announces its finished items, waits until all items of the layer are finished, and merges the pages of
            // its share of the (row, query head) pairs.
            int total_items = 0;
            for (int rg = 0; rg < RG; ++rg) total_items += (p.row_pos[rg * ANPD_ROWS + ANPD_ROWS - 1] / KV_PAGE + 1) * p.Hkv;
            group_bar();
            if (e == 0) {
                if (n_mine > 0) red_add_release(sync_at(l, p.o_ditems), n_mine);
                if (!fwait(sync_at(l, p.o_ditems), total_items)) *abortp = 1;
            }
            group_bar();
            if (*abortp) return false;
            int n_units = 0;
            for (int u = cta; u < rows * p.Hq; u += G) { combine_unit(u / p.Hq, u % p.Hq); ++n_units; }
            if (n_units > 0) {
                fence_async_global();
                group_bar();
                if (e == 0) red_add_release(sync_at(l, p.o_dao), n_units);
            }
            return true;
        };

        // optional time stamps of CTA 0's epilogue group at the end of every phase (a debugging aid)
        auto stamp = [&](int slot) {
            if (p.trace && cta == p.trace_cta && e == 0) {
                unsigned long long t;
                asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
                p.trace[slot] = t;
            }
        };
        stamp(0);
        // embedding: tile t of the residual stream by CTA t
        for (int tile = cta; tile < d_tiles; tile += G) {
            resid_tail(tile, nullptr, p.layers[0].attn_norm, p.imgA, p.ssA);
            publish(sync_at(0, p.o_dh));
            group_bar();
        }
        for (int l = 0; l < p.L && ok; ++l) {
            ok = epi_gemm(GK_QKV, l); stamp(1 + 5 * l);
            ok = ok && epi_attn(l); stamp(2 + 5 * l);
            ok = ok && epi_gemm(GK_O, l); stamp(3 + 5 * l);
            ok = ok && epi_gemm(GK_GU, l); stamp(4 + 5 * l);
            ok = ok && epi_gemm(GK_DOWN, l); stamp(5 + 5 * l);
        }
        ok = ok && epi_gemm(GK_LM, p.L);
        stamp(1 + 5 * p.L);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)tmem_cols) : "memory");
    }
    if (threadIdx.x == 0 && abort_flag) atomicExch(p.err, ST_ERR_TIMEOUT);
}

inline size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }

}  // namespace

bool step_kernel_eligible(const anpd_model* m, const anpd_kv* kv) {
    const anpd_model_config& c = m->cfg;
    // Opt-in (ANPD_STEP_KERNEL=1): measured at the 7B shape the step takes 4.0 ms in this kernel against 3.2 ms as a chain
    // of kernels - handing a projection's result to the next one through global memory (partial sums, arrival counter,
    // tail, phase counter, operand fetch: five to seven dependent round trips, each slow while the rings prefetch) costs
    // more than the kernel boundaries it replaces.
    if (std::getenv("ANPD_STEP_KERNEL") == nullptr || m->plain_gemm) return false;
    if (c.head_dim != 128 || c.n_q_heads != c.n_kv_heads) return false;
    if (c.d_model % TILE || c.d_ffn % TILE) return false;
    if (kv->batch * ANPD_ROWS > 64 || kv->pages_per_seq > ST_MAX_PAGES) return false;
    if (!kv->attn_tc) return false;
    for (int k = 0; k < GK_COUNT; ++k) if (m->plan[k].max_segs > MAX_SEGS) return false;
    return true;
}

anpd_status step_kernel_setup(anpd_model* m, anpd_kv* kv) {
    const anpd_model_config& c = m->cfg;
    Workspace& ws = kv->ws;
    StepParams& p = kv->step;
    kv->step_ready = false;
    kv->step_slab = nullptr;
    if (!step_kernel_eligible(m, kv)) return ANPD_OK;
    const int rows = kv->batch * ANPD_ROWS, NR = 2 * rows;
    const int d_tiles = c.d_model / TILE, f_tiles = c.d_ffn / TILE, RG = kv->batch;
    // shared memory: the ring takes what the fixed buffers leave
    int dev = 0, max_smem = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    CUDA_TRY(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    const int scratch_bytes = std::max(SCRATCH_MIN, (int)up256((size_t)d_tiles * rows * 4));
    const int fixed = 1024 + 2 * QP_BYTES + scratch_bytes + 4096 /* static barriers and reduction scratch */;
    const int stage_bytes = SB * (W_BYTES + NR * 128);
    int stages = std::min(ST_MAX_STAGES, (max_smem - fixed) / stage_bytes);
    if (const char* s = std::getenv("ANPD_STEP_STAGES")) stages = std::max(2, std::min(stages, std::atoi(s)));
    if (stages < 2) return ANPD_OK;
    kv->step_smem = 1024 + stages * stage_bytes + 2 * QP_BYTES + scratch_bytes;

    // buffers only this path uses
    size_t part_bytes[GK_COUNT], total = 0;
    for (int k = 0; k < GK_COUNT; ++k) {
        const GemmPlan& pl = m->plan[k];
        part_bytes[k] = up256((size_t)pl.max_segs * rows * (size_t)pl.m_tiles * TILE * 4);
        total += part_bytes[k];
    }
    const size_t b_ss = up256((size_t)d_tiles * rows * 4);
    auto img_bytes = [&](int K) { return up256((size_t)((K + 63) / 64) * NR * 128); };
    const size_t b_imgd = img_bytes(c.d_model), b_imgq = img_bytes(m->dq), b_imgf = img_bytes(c.d_ffn);
    const int lm_tiles = m->plan[GK_LM].m_tiles;
    const size_t b_amax = up256((size_t)rows * lm_tiles * 4);
    // per layer: five phase counters, each in a 128-byte line of its own (they are polled), then the tiles' arrival counters
    int off = 0;
    p.o_dh = off; off += 32;
    p.o_dqkv = off; off += 32;
    p.o_dao = off; off += 32;
    p.o_dhB = off; off += 32;
    p.o_dact = off; off += 32;
    p.o_ditems = off; off += 32;
    p.o_cqkv = off; off += m->plan[GK_QKV].m_tiles;
    p.o_cattn = off; off += c.n_kv_heads * RG;
    p.o_co = off; off += d_tiles;
    p.o_cgu = off; off += f_tiles;
    p.o_cdown = off; off += d_tiles;
    p.o_clm = off; off += lm_tiles;
    off = (off + 31) / 32 * 32;
    p.sync_stride = off;
    kv->step_sync_bytes = (size_t)(c.n_layers + 1) * off * sizeof(int);
    const size_t b_sync = up256(kv->step_sync_bytes), b_layers = up256(sizeof(StepLayer) * (size_t)c.n_layers);
    const bool want_trace = std::getenv("ANPD_STEP_TRACE") != nullptr;
    const size_t b_trace = want_trace ? up256((size_t)(29 * c.n_layers + 2) * 8) : 0;
    total += 2 * b_imgd + b_imgq + b_imgf + 2 * b_ss + 2 * b_amax + b_sync + b_layers + b_trace;
    if (cudaMalloc(&kv->step_slab, total) != cudaSuccess) { cudaGetLastError(); kv->step_slab = nullptr; return ANPD_ERR_OOM; }
    CUDA_TRY(cudaMemsetAsync(kv->step_slab, 0, total, m->stream));
    char* q = (char*)kv->step_slab;
    auto take = [&](size_t bytes) { void* r = q; q += bytes; return r; };
    for (int k = 0; k < GK_COUNT; ++k) {
        const GemmPlan& pl = m->plan[k];
        StepGemm& g = p.g[k];
        g.N = pl.N; g.K = pl.K; g.m_tiles = pl.m_tiles; g.k_blocks = pl.k_blocks; g.grid = pl.grid;
        g.first_cta = pl.d_first_cta; g.seg_count = pl.d_seg_count;
        g.part = (float*)take(part_bytes[k]);
        g.ld_part = pl.m_tiles * TILE;
        g.seg_stride = (unsigned long long)rows * g.ld_part;
    }
    p.imgA = (unsigned char*)take(b_imgd); p.imgB = (unsigned char*)take(b_imgd);
    p.img_ao = (unsigned char*)take(b_imgq); p.img_act = (unsigned char*)take(b_imgf);
    p.ssA = (float*)take(b_ss); p.ssB = (float*)take(b_ss);
    p.amax_val = (float*)take(b_amax); p.amax_idx = (int*)take(b_amax);
    p.sync = (int*)take(b_sync);
    StepLayer* d_layers = (StepLayer*)take(b_layers);
    p.trace = want_trace ? (unsigned long long*)take(b_trace) : nullptr;
    p.trace_cta = want_trace ? std::max(0, std::min(m->num_sms - 1, std::atoi(std::getenv("ANPD_STEP_TRACE")))) : 0;
    std::vector<StepLayer> hl(c.n_layers);
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerW& w = m->layers[l];
        hl[l] = StepLayer{w.wqkv, w.wo, w.wgu, w.wd, w.attn_norm, w.ffn_norm};
    }
    CUDA_TRY(cudaMemcpyAsync(d_layers, hl.data(), sizeof(StepLayer) * hl.size(), cudaMemcpyHostToDevice, m->stream));
    CUDA_TRY(cudaStreamSynchronize(m->stream));
    p.layers = d_layers;
    p.map_k = kv->map_k; p.map_v = kv->map_v;
    p.embed = m->embed; p.lm_head = m->lm_head; p.final_norm = m->final_norm;
    p.L = c.n_layers; p.d = c.d_model; p.F = c.d_ffn; p.V = c.vocab; p.Hq = c.n_q_heads; p.Hkv = c.n_kv_heads; p.hd = c.head_dim;
    p.dq = m->dq; p.rows = rows; p.stages = stages;
    p.eps = c.rms_eps; p.q_scale = 1.4426950408889634f / sqrtf((float)c.head_dim);
    p.row_tok = ws.row_tok; p.row_pos = ws.row_pos; p.row_seq = ws.row_seq; p.row_ok = ws.row_ok;
    p.x = ws.x;
    p.q_hi = ws.q_hi; p.q_lo = ws.q_lo;
    p.pm = ws.attn_m; p.pl = ws.attn_l; p.po = ws.attn_o;
    p.logits = ws.logits;
    p.kpool = kv->kpool; p.vpool = kv->vpool;
    p.layer_elems = (unsigned long long)kv->total_pages * c.n_kv_heads * KV_PAGE * c.head_dim;
    p.layer_rows = kv->total_pages * c.n_kv_heads * KV_PAGE;
    p.page_table = kv->page_table; p.pages_per_seq = kv->pages_per_seq;
    p.rope_cos = kv->rope_cos; p.rope_sin = kv->rope_sin;
    p.err = ws.gemm_err;
    kv->step_ready = true;
    return ANPD_OK;
}

// ANPD_STEP_TRACE=1: prints, for the last step the kernel ran, how long CTA 0's epilogue group spent in each phase.
void step_kernel_trace_dump(anpd_kv* kv) {
    if (!kv->step_ready || !kv->step.trace) return;
    const int L = kv->step.L, n = 5 * L + 2;
    std::vector<unsigned long long> t(n);
    if (cudaMemcpy(t.data(), kv->step.trace, sizeof(unsigned long long) * n, cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return; }
    if (t[n - 1] <= t[0]) return;
    double ph[5] = {0, 0, 0, 0, 0};
    for (int l = 0; l < L; ++l)
        for (int k = 0; k < 5; ++k) ph[k] += (double)(t[1 + 5 * l + k] - t[5 * l + k]) * 1e-3;
    std::fprintf(stderr, "[anpd] step kernel, CTA %d, mean us per layer: QKV %.2f  attention %.2f  O %.2f  gate/up %.2f  down %.2f;  LM head %.2f;  step %.1f\n",
                 kv->step.trace_cta, ph[0] / L, ph[1] / L, ph[2] / L, ph[3] / L, ph[4] / L, (double)(t[n - 1] - t[n - 2]) * 1e-3, (double)(t[n - 1] - t[0]) * 1e-3);
    // per projection: from the end of the previous phase's epilogue to the input being announced, to the first MMA, to the
    // last MMA issued, to the end of this phase's epilogue (tail included)
    std::vector<unsigned long long> u((size_t)12 * L);
    if (cudaMemcpy(u.data(), kv->step.trace + n, sizeof(unsigned long long) * u.size(), cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return; }
    std::vector<unsigned long long> w((size_t)12 * L);
    if (cudaMemcpy(w.data(), kv->step.trace + n + 12 * L, sizeof(unsigned long long) * w.size(), cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return; }
    const char* names[4] = {"QKV", "O", "gate/up", "down"};
    const int epi_end[4] = {1, 3, 4, 5}, prev_end[4] = {0, 2, 3, 4};
    for (int g = 0; g < 4; ++g) {
        double a = 0, b = 0, c2 = 0, d2 = 0;
        for (int l = 1; l < L; ++l) {
            const unsigned long long* q = &u[(size_t)(l * 4 + g) * 3];
            a += (double)((long long)q[0] - (long long)t[5 * l + prev_end[g]]) * 1e-3;
            b += (double)((long long)q[1] - (long long)q[0]) * 1e-3;
            c2 += (double)((long long)q[2] - (long long)q[1]) * 1e-3;
            d2 += (double)((long long)t[5 * l + epi_end[g]] - (long long)q[2]) * 1e-3;
        }
        const int cnt = L > 1 ? L - 1 : 1;
        double ww = 0, wa = 0, wc = 0;
        for (int l = 1; l < L; ++l) { ww += (double)w[(size_t)(l * 4 + g) * 3]; wa += (double)w[(size_t)(l * 4 + g) * 3 + 1]; wc += (double)w[(size_t)(l * 4 + g) * 3 + 2]; }
        std::fprintf(stderr, "[anpd]   %-8s prev epilogue end -> input announced %.2f -> first MMA %.2f -> last MMA issued %.2f -> epilogue end %.2f"
                             ";  MMA thread waited (kcycles) stage %.1f  (%.1f)  accumulator %.1f\n",
                     names[g], a / cnt, b / cnt, c2 / cnt, d2 / cnt, ww / cnt * 1e-3, wa / cnt * 1e-3, wc / cnt * 1e-3);
    }
}

anpd_status step_kernel_enqueue(anpd_model* m, anpd_kv* kv, int max_pos, bool want_logits) {
    static int smem_set[64] = {0};                      // largest dynamic shared memory size set so far, per device
    if (m->device >= 0 && m->device < 64 && smem_set[m->device] < kv->step_smem) {
        CUDA_TRY(cudaFuncSetAttribute(step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kv->step_smem));
        smem_set[m->device] = kv->step_smem;
    }
    Workspace& ws = kv->ws;
    const int chunks = max_pos / KV_PAGE + 1;
    CUDA_TRY(cudaMemsetAsync(kv->step.sync, 0, kv->step_sync_bytes, m->stream));
    LAUNCH(&m->prof, m->stream, KC_GEMM, m->streamed_bytes,
           (launch_k(step_kernel, m->num_sms, ST_THREADS, (size_t)kv->step_smem, m->stream, kv->step, chunks, want_logits ? 1 : 0)));
    CUDA_TRY(cudaGetLastError());
    ws.amax_nblk = m->plan[GK_LM].m_tiles;             // the argmax candidates are per 128-feature tile, in this path's own arrays
    ws.amax_val_use = kv->step.amax_val;
    ws.amax_idx_use = kv->step.amax_idx;
    return ANPD_OK;
}
