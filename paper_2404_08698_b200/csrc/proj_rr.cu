// Projections of a single-sequence verify step (8 rows) with everything that follows them fused in:
//   QKV     -> rotary embedding, query scaling, K/V rows appended to the paged cache
//   O, down -> residual add, the next RMSNorm's gain, the row's sum of squares (partial)
//   gate/up -> SwiGLU
//   LM head -> logits (optional) and the per-CTA argmax
// (paper Section 3.1, "Verification": the forward over the K+1 tokens of a step.)
//
// The step is bound by reading every weight once.  Each of the G = #SMs CTAs owns a contiguous range
// of OUTPUT FEATURES of the matrix (r = about N / G weight rows) and walks the whole contraction
// dimension, so a CTA ends with complete dot products and finishes the layer's elementwise work in
// its epilogue: no partial sums cross CTAs, and the small kernels that would sit between two
// projections (each a dependent launch with its own memory round trip) do not exist.
//
// How the product maps onto tcgen05.mma.  One instruction (M = 128, K = 16) costs max(45, N / 2)
// cycles whatever M holds, so to stay bound by memory every instruction must consume several KB of
// weights; a CTA's r rows (28 for a 4096-wide output on 148 SMs) x 16 inputs are far too little.
// The weights are therefore the N operand, and P consecutive 16-wide slices of K are packed into ONE
// instruction: its N rows are (slice p, feature f), P * r <= 256 of them, each a 32-byte row; its M
// rows are (slice p, activation row), 16 per slice (8 hi terms, 8 lo terms).  The instruction
// computes every slice of the activations against every slice of the weights; the blocks with equal
// slice index are the wanted partial dot products, the others are ignored.  P * r * 32 bytes of
// weights per instruction: 7 KB for r = 28, P = 8.  The epilogue adds, per feature and row, the 2 P
// accumulator lanes (hi and lo term of every slice) in a fixed order.
//
// Storage.  Per CTA the weights are the exact shared-memory image of its instructions' N operands
// (32-byte rows, 32-byte swizzle), step after step, stage after stage, the stages of all CTAs side by
// side: at any time the G CTAs read one contiguous window that sweeps through memory.  The activations
// arrive as a ready-made operand image too (written by the producing epilogue): per 64-wide k-block
// 64 rows (slice, activation row) of 32 bytes = 2 KB, one linear bulk copy per stage.
//
// RMSNorm is deferred: the producer of the residual stream writes x * gain (hi + lo) and each CTA's
// partial sum of squares; the consuming projection multiplies its outputs by 1 / rms(x), which
// commutes with the matrix product.  Partial sums are added in CTA order: the same bits in every launch.
// Features are permuted at model creation so that the two members of a rotary pair (dimension i and
// i + head_dim/2) and of a SwiGLU pair (gate j, up j) are neighbours; a CTA's range starts at an even
// feature, so a pair is exchanged with one shuffle.
#include "internal.h"
#include "tc_ptx.cuh"

#include <math_constants.h>

#include <algorithm>
#include <cstdlib>

typedef __nv_bfloat16 bf16;

namespace {

using namespace tc;

constexpr int RR_THREADS = 192;          // warp 0: producer, warp 1: MMA issuer + TMEM owner, warps 2-5: epilogue
constexpr int RR_MAX_STAGES = 16;
constexpr int RR_ERR_TIMEOUT = 203;
constexpr int A_KB_BYTES = 2048;         // one k-block of the activation operand: 4 slices x (8 hi + 8 lo rows) x 32 bytes
constexpr int RR_MAX_STEPS = 4;          // most MMAs a stage may hold (rr_make_plan sizes the stages accordingly)
constexpr int RR_TMEM_COLS = 256;        // accumulator: up to 256 (slice, feature) columns

struct RRArgs {
    const unsigned char* w;              // this matrix in row-range storage
    const unsigned char* act;            // activation operand image, A_KB_BYTES per k-block
    int N;                               // output features (valid)
    int pairs;                           // feature pairs = ceil(N / 2), cut evenly across the grid
    int r_max;                           // most features a CTA owns
    int P;                               // 16-wide slices of K per instruction
    int k_blocks, kb, n_stages, stages;
    int w_step_stride;                   // shared-memory bytes between the weight operands of two steps of a stage
    int w_step_global;                   // the same in the stored image (P * r_max * 32)
    int a_off;                           // offset of the activation tiles inside a stage
    int stage_bytes;
    int scratch_off;                     // epilogue scratch behind the ring (and its read-ahead slack)
    int rotate;                          // CTAs start their walk over K at different stages (see rr_rotation)
    int one_copy;                        // a stage's weights are fetched by one copy (rows up to r_max included)
    unsigned long long slot_bytes;       // global bytes per (stage, CTA)
    int* err;
};

struct RREpi {
    // input normalisation (QKV, gate/up, LM head): rstd[row] = rsqrt(sum_i ss_in[i][row] / d_in + eps)
    const float* ss_in; int n_parts_in; float inv_d_in; float eps;
    // QKV
    const int* row_pos; const int* row_seq; const int* row_ok; const float* rope_cos; const float* rope_sin;
    const int* page_table; int pages_per_seq; int Hq, Hkv, hd; float q_scale;
    bf16* q_hi; bf16* q_lo; bf16* kpool_l; bf16* vpool_l;
    // O / down
    float* x; const float* gain; float* ss_out; int d;
    // O / down / gate-up: operand image of the next projection
    unsigned char* act_out;
    // LM head
    float* logits; float* amax_val; int* amax_idx; int V;
    // plain product (test hook): out[row][n]
    float* raw_out;
};

__device__ __forceinline__ void split_store(unsigned char* img, int row, int k, float v) {
    const bf16 hi = __float2bfloat16_rn(v);
    const bf16 lo = __float2bfloat16_rn(v - __bfloat162float(hi));
    *(bf16*)(img + act_img_offset(row, k)) = hi;
    *(bf16*)(img + act_img_offset(ANPD_ROWS + row, k)) = lo;
}

// Shared-memory operand descriptor: K-major tile of 32-byte rows, 32-byte swizzle, groups of 8 rows 256 bytes apart.
__device__ __forceinline__ uint64_t make_smem_desc_sw32(uint32_t saddr) {
    uint64_t d = (uint64_t)((saddr >> 4) & 0x3FFFu);
    d |= (uint64_t)1 << 16;               // leading byte offset (unused: K extent = one swizzle row)
    d |= (uint64_t)(256 >> 4) << 32;      // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;               // descriptor version of this architecture
    d |= (uint64_t)6 << 61;               // 32-byte swizzle
    return d;
}

// One MMA, issued only if `enable`; the operand descriptors are given as (low word, high word): all the per-step
// arithmetic happens on the low words, which hold the operand's shared-memory address.
__device__ __forceinline__ void tc_mma_bf16_lo(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc, uint32_t accumulate,
                                               uint32_t enable) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "setp.ne.b32 q, %6, 0;\n\t"
        "mov.b64 da, {%1, %3};\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, {%7, %7, %7, %7}, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate), "r"(enable), "r"(0u) : "memory");
}

__device__ __forceinline__ void tc_ld8(uint32_t taddr, float* v) {
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]) : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float* v) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]),
          "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
          "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]),
          "=r"(r[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_ld2(uint32_t taddr, float* v) {
    uint32_t r[2];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0, %1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
    v[0] = __uint_as_float(r[0]);
    v[1] = __uint_as_float(r[1]);
}

// The image offset of element (term row, k) is  k-part + 32 * row + 16 * (chunk(k) ^ swizzle(row)),  and swizzle(row) is
// bit 2 of the row: the k-part with either chunk position is computed once per feature, the row part is a constant.
struct ImgCol { uint32_t off[2]; };          // offset of (row with swizzle bit 0 / 1, k) minus the row's own 32 * row
__device__ __forceinline__ ImgCol img_col(int k) {
    const uint32_t base = (uint32_t)(k >> 6) * 2048u + (uint32_t)((k >> 4) & 3) * 512u + (uint32_t)(k & 7) * 2u;
    const uint32_t chunk = (uint32_t)(k >> 3) & 1u;
    ImgCol c;
    c.off[0] = base + (chunk << 4);
    c.off[1] = base + ((chunk ^ 1u) << 4);
    return c;
}
__device__ __forceinline__ void split_store_row(unsigned char* img, const ImgCol& c, int row, float v) {
    const bf16 hi = __float2bfloat16_rn(v);
    const bf16 lo = __float2bfloat16_rn(v - __bfloat162float(hi));
    *(bf16*)(img + c.off[(row >> 2) & 1] + row * 32) = hi;                                   // term row `row` (hi part)
    *(bf16*)(img + c.off[((ANPD_ROWS + row) >> 2) & 1] + (ANPD_ROWS + row) * 32) = lo;       // term row 8 + row (lo part)
}
template <int ROW>
__device__ __forceinline__ void split_store_at(unsigned char* img, const ImgCol& c, float v) {
    const bf16 hi = __float2bfloat16_rn(v);
    const bf16 lo = __float2bfloat16_rn(v - __bfloat162float(hi));
    *(bf16*)(img + c.off[(ROW >> 2) & 1] + ROW * 32) = hi;                                   // term row ROW (hi part)
    *(bf16*)(img + c.off[((ANPD_ROWS + ROW) >> 2) & 1] + (ANPD_ROWS + ROW) * 32) = lo;       // term row 8 + ROW (lo part)
}
template <int ROW = 0>
__device__ __forceinline__ void split_store_rows(unsigned char* img, const ImgCol& c, const float* v) {
    split_store_at<ROW>(img, c, v[ROW]);
    if constexpr (ROW + 1 < ANPD_ROWS) split_store_rows<ROW + 1>(img, c, v);
}

template <int EPI, int MT>
__global__ void __launch_bounds__(RR_THREADS, 1) proj_rr_kernel(const RRArgs g, const RREpi e) {
    extern __shared__ __align__(1024) unsigned char rr_smem_raw[];
    __shared__ uint64_t bar_full[RR_MAX_STAGES], bar_empty[RR_MAX_STAGES], bar_done;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag, mma_ok;
    __shared__ float red_f[4][ANPD_ROWS], s_rstd[ANPD_ROWS];
    __shared__ int red_i[4][ANPD_ROWS], s_pos[ANPD_ROWS], s_page[ANPD_ROWS];

    pdl_trigger();
    unsigned char* smem = rr_smem_raw + ((1024u - (smem_u32(rr_smem_raw) & 1023u)) & 1023u);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, c = blockIdx.x;
    const int start = 2 * (int)((long long)c * g.pairs / G);
    const int r = 2 * (int)((long long)(c + 1) * g.pairs / G) - start;          // features of this CTA
    const int P = g.P;
    // Every CTA needs every k-block of the activations.  If all walked K in the same order, all SMs would ask for the
    // same 2 KB of the activation image at the same moment; each CTA therefore starts at its own stage and wraps
    // around.  The weights are stored in the order their CTA reads them.
    const int rot = g.rotate ? rr_rotation(c, G, g.n_stages) : 0;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < g.stages; ++s) { mbar_init(&bar_full[s], 1); mbar_init(&bar_empty[s], 1); }
        mbar_init(&bar_done, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"((uint32_t)RR_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *((volatile uint32_t*)&tmem_base_slot);
    volatile int* abortp = &abort_flag;
    // The producer and the MMA issuer are single threads whose loop body runs once per stage: at one dependent
    // instruction every few cycles, a division or a 64-bit product per stage already costs more time than the stage's
    // bytes take to arrive.  Everything that varies per stage is therefore advanced by additions.  Only the last stage
    // of K (in logical order; this CTA meets it at turn tail_turn of its rotated walk) can hold fewer k-blocks.
    const int tail_kb = g.k_blocks - (g.n_stages - 1) * g.kb;                    // k-blocks of the last logical stage
    const int steps_full = (g.kb * 4 + P - 1) / P, steps_tail = (tail_kb * 4 + P - 1) / P;
    const int tail_turn = g.n_stages - 1 - rot;                                  // turn at which the slot holds the last logical stage

    if (warp == 0) {
        // ---------------- producer (one warp: lane 0 keeps the barriers, lanes 0.. issue one weight copy each, lane 31 the activations) ----------------
        const uint64_t pol_w = policy_evict_first(), pol_a = policy_evict_last();
        const uint32_t w_step_bytes = (uint32_t)(P * r) * 32u;                   // this CTA's rows of one step
        const uint32_t w_copy = g.one_copy ? (uint32_t)g.w_step_global : w_step_bytes;
        // an instruction that packs eight slices spans two k-blocks: whole steps are fetched (the image ends with a zero k-block)
        const uint32_t a_full = (uint32_t)g.kb * A_KB_BYTES, a_tail = (uint32_t)(P == 8 ? (tail_kb + 1) & ~1 : tail_kb) * A_KB_BYTES;
        const uint32_t tx_full = (uint32_t)steps_full * w_copy + a_full, tx_tail = (uint32_t)steps_tail * w_copy + a_tail;
        const unsigned long long src_turn = (unsigned long long)G * g.slot_bytes;                       // from one turn's slot to the next
        // The warp stays converged: every lane runs the same straight line per stage, and the copies are predicated
        // instructions (lane 0: the barrier's byte count; lanes below the stage's step count: one weight copy each, or
        // lane 0 alone when a stage is one copy; lane 31: the activations).  Per-lane constants:
        const unsigned char* w_src = g.w + (unsigned long long)c * g.slot_bytes + (g.one_copy ? 0 : (size_t)lane * g.w_step_global);
        const uint32_t lane_dst = g.one_copy ? 0u : (uint32_t)lane * (uint32_t)g.w_step_stride;
        const uint32_t wb_full = g.one_copy ? (uint32_t)steps_full * w_copy : w_step_bytes, wb_tail = g.one_copy ? (uint32_t)steps_tail * w_copy : w_step_bytes;
        const uint32_t wen_full = g.one_copy ? (lane == 0) : (lane < steps_full), wen_tail = g.one_copy ? (lane == 0) : (lane < steps_tail);
        const uint32_t is0 = lane == 0, is31 = lane == 31;
        const unsigned char* a_src = g.act + (size_t)rot * a_full;                                       // activations of the first turn's stage
        const unsigned char* const a_wrap = g.act + (size_t)g.n_stages * a_full;
        auto load_w = [&](int turn, uint32_t dst, uint32_t bar) {
            const bool tail = turn == tail_turn;
            asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %2, 0;\n\t@p mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n\t}"
                         ::"r"(bar), "r"(tail ? tx_tail : tx_full), "r"(is0) : "memory");
            __syncwarp();
            asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                         "@p cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;\n\t}"
                         ::"r"(dst + lane_dst), "l"(w_src), "r"(tail ? wb_tail : wb_full), "r"(bar), "l"(pol_w), "r"(tail ? wen_tail : wen_full) : "memory");
            w_src += src_turn;
        };
        auto load_a = [&](int turn, uint32_t dst, uint32_t bar) {
            asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                         "@p cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;\n\t}"
                         ::"r"(dst + (uint32_t)g.a_off), "l"(a_src), "r"(turn == tail_turn ? a_tail : a_full), "r"(bar), "l"(pol_a), "r"(is31) : "memory");
            a_src += a_full;
            a_src = a_src == a_wrap ? g.act : a_src;
        };
        // the weights depend on no earlier kernel: fill the ring first, then wait for the activations' producer
        const uint32_t ring = smem_u32(smem);
        const int ahead = min(g.stages, g.n_stages);
        for (int s = 0; s < ahead; ++s) load_w(s, ring + (uint32_t)s * (uint32_t)g.stage_bytes, smem_u32(&bar_full[s]));
        pdl_wait();
        for (int s = 0; s < ahead; ++s) load_a(s, ring + (uint32_t)s * (uint32_t)g.stage_bytes, smem_u32(&bar_full[s]));
        int stage = ahead % g.stages;
        uint32_t phase = (ahead == g.stages) ? 1u : 0u;
        uint32_t dst = ring + (uint32_t)stage * (uint32_t)g.stage_bytes;
        int issued = ahead;
        bool ok = true;
        for (int s = ahead; s < g.n_stages; ++s) {
            ok = mbar_wait(&bar_empty[stage], phase ^ 1u, abortp);
            if (!ok) break;
            const uint32_t bar = smem_u32(&bar_full[stage]);
            load_w(s, dst, bar);
            load_a(s, dst, bar);
            ++issued;
            dst += (uint32_t)g.stage_bytes;
            if (++stage == g.stages) { stage = 0; phase ^= 1u; dst = ring; }
        }
        if (!ok && lane == 0) {
            // gave up: let every copy already issued land before the CTA may exit
            const int n = issued < g.stages ? issued : g.stages;
            for (int i = 0; i < n; ++i) {
                const int idx = issued - 1 - i;
                const int st = idx % g.stages;
                const uint32_t ph = (uint32_t)((idx / g.stages) & 1);
                for (unsigned spin = 0; spin < WAIT_LIMIT && !mbar_try_wait(&bar_full[st], ph); ++spin) {}
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        pdl_wait();                                       // nothing to multiply before the activations exist: sleep instead of polling
        if (lane == 0) {
            // fp32 accumulate, bf16 x bf16, both operands K-major, M = 128 (16 P real rows), N = P * r rounded up to 16
            const int Nmma = (P * r + 15) & ~15;
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(Nmma >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
            // Every operand sits at a multiple of 256 bytes from the ring's start, so its descriptor is the ring's with a
            // constant added to the low word (the 16-byte-unit address field; the ring lies below 256 KB, no carry out of it).
            // This thread is the warp's only active lane: every branch costs it a divergence bracket of dozens of cycles,
            // and a dependent instruction chain a few cycles per link.  The MMAs of a stage are therefore issued as one
            // straight line of predicated instructions (steps beyond the stage's count are switched off), not as a loop.
            const uint64_t desc0 = make_smem_desc_sw32(smem_u32(smem));
            const uint32_t lo0 = (uint32_t)desc0, hi = (uint32_t)(desc0 >> 32);
            const uint32_t stage_step = (uint32_t)(g.stage_bytes >> 4), w_step = (uint32_t)(g.w_step_stride >> 4);
            const uint32_t a_step = (uint32_t)((P * 512) >> 4), a_off = (uint32_t)(g.a_off >> 4);
            uint32_t d_stage = lo0;
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            uint32_t acc = 0;
            for (int s = 0; s < g.n_stages; ++s) {
                ok = mbar_wait(&bar_full[stage], phase, abortp);
                if (!ok) break;
                tc_fence_after();
                const int n_steps = s == tail_turn ? steps_tail : steps_full;
#pragma unroll
                for (int t = 0; t < RR_MAX_STEPS; ++t) {      // A: (slice, activation row) x 16; B: (slice, feature) x 16
                    tc_mma_bf16_lo(tmem_base, d_stage + a_off + (uint32_t)t * a_step, d_stage + (uint32_t)t * w_step, hi, idesc,
                                   t == 0 ? acc : 1u, t < n_steps ? 1u : 0u);
                }
                acc = 1;
                tc_commit(&bar_empty[stage]);                   // frees the stage once these MMAs have read it
                d_stage += stage_step;
                if (++stage == g.stages) { stage = 0; phase ^= 1u; d_stage = lo0; }
            }
            if (ok) {
                tc_commit(&bar_done);
                ok = mbar_wait(&bar_done, 0, abortp);     // one thread polls; the epilogue warps sleep at the hardware barrier below
            }
            mma_ok = ok ? 1 : 0;
        }
        __syncwarp();
        asm volatile("bar.sync 2, 160;" ::: "memory");    // accumulators complete: release the four epilogue warps
    } else {
        // ---------------- epilogue warps ----------------
        const int quad = warp & 3;                        // a warp may only touch TMEM lanes 32 * (warp % 4) .. + 31
        const int ew = warp - 2;                          // 0..3
        const int et = ew * 32 + lane;                    // 0..127: thread et finishes features et, et + 128 of the CTA's range
        pdl_wait();
        // Work that needs no accumulator, done while the weights stream.  What the row loop below needs per row or per
        // (feature, row) is parked in shared memory (a scratch area behind the ring), so that the loop can stay rolled:
        // the epilogue runs once per launch, its code is fetched cold, and eight unrolled copies of it cost more in
        // instruction fetches than they save in arithmetic.
        float* scratch = (float*)(smem + g.scratch_off);              // [2][8][r] rotary factors (QKV) or [8][r] residual (O, down)
        if (EPI == RR_QKV || EPI == RR_GU || EPI == RR_LM) {
            if (ew == 0) {
#pragma unroll 1
                for (int row = 0; row < ANPD_ROWS; ++row) {
                    float sq = 0.0f;
                    for (int i = lane; i < e.n_parts_in; i += 32) sq += e.ss_in[i * ANPD_ROWS + row];
                    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
                    if (lane == 0) s_rstd[row] = rsqrtf(sq * e.inv_d_in + e.eps);
                }
            }
        }
        if (EPI == RR_QKV) {
            if (et < ANPD_ROWS) {
                const int pos = e.row_pos[et];
                s_pos[et] = pos;
                s_page[et] = e.row_ok[et] ? e.page_table[e.row_seq[et] * e.pages_per_seq + pos / KV_PAGE] : -1;
            }
            const int half = e.hd >> 1;
            for (int idx = et; idx < ANPD_ROWS * r; idx += 128) {
                const int row = idx / r, i = idx - row * r, n = start + i;
                const int head = n / e.hd, pp = (n - head * e.hd) >> 1;
                const bool rot_here = n < g.N && head < e.Hq + e.Hkv;
                const int pos = e.row_pos[row];
                scratch[idx] = rot_here ? e.rope_cos[(size_t)pos * half + pp] : 1.0f;
                scratch[ANPD_ROWS * r + idx] = rot_here ? e.rope_sin[(size_t)pos * half + pp] : 0.0f;
            }
        }
        if (EPI == RR_RESID) {
            for (int idx = et; idx < ANPD_ROWS * r; idx += 128) {
                const int row = idx / r, n = start + idx - row * r;
                scratch[idx] = n < g.N ? e.x[(size_t)row * e.d + n] : 0.0f;
            }
        }
        asm volatile("bar.sync 2, 160;" ::: "memory");    // the MMA warp arrives once every accumulator is complete (or it gave up)
        const bool ok = *((volatile int*)&mma_ok) != 0;
        tc_fence_after();
        // Accumulator lane (slice p, term/row a) holds, in columns [p * r, p * r + r), that slice's share of the dot
        // products of activation term a with the CTA's features.  Stage them in shared memory (the ring is idle now:
        // every copy has landed and every MMA has read its operands) as tr[lane][feature].
        float* tr = (float*)smem;
        const int tr_stride = r | 1;
        if (ok) {
            for (int gsel = 0; gsel < 2; ++gsel) {
                const int p = 2 * quad + gsel;                         // the slice of this warp's lanes 16 gsel .. 16 gsel + 15
                if (p >= P) break;
                const bool mine = (lane >> 4) == gsel;
                float* dst = tr + (size_t)(quad * 32 + lane) * tr_stride;
                const uint32_t t0 = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(p * r);
                int f = 0;
                for (; f + 32 <= r; f += 32) {
                    float v[32];
                    tc_ld32(t0 + (uint32_t)f, v);
                    if (mine)
#pragma unroll
                        for (int u = 0; u < 32; ++u) dst[f + u] = v[u];
                }
                for (; f + 8 <= r; f += 8) {
                    float v[8];
                    tc_ld8(t0 + (uint32_t)f, v);
                    if (mine)
#pragma unroll
                        for (int u = 0; u < 8; ++u) dst[f + u] = v[u];
                }
                for (; f < r; f += 2) {
                    float v[2];
                    tc_ld2(t0 + (uint32_t)f, v);
                    if (mine) { dst[f] = v[0]; dst[f + 1] = v[1]; }
                }
            }
        }
        tc_fence_before();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (ok) {
            // per-feature constants of this thread's (up to MT) features
            int nn[MT];
            bool valid[MT];
            ImgCol col[MT];
            float gn[MT];
            int head[MT], dim[MT], sec[MT];
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                const int i = m * 128 + et;
                nn[m] = start + i;
                valid[m] = i < r && nn[m] < g.N;
                gn[m] = 0.0f; head[m] = 0; dim[m] = 0; sec[m] = 0;
                if (EPI == RR_RESID) { col[m] = img_col(nn[m]); gn[m] = valid[m] ? e.gain[nn[m]] : 0.0f; }
                if (EPI == RR_GU) col[m] = img_col(nn[m] >> 1);
                if (EPI == RR_QKV) {
                    const int half = e.hd >> 1;
                    head[m] = nn[m] / e.hd;
                    const int p = nn[m] - head[m] * e.hd;
                    sec[m] = p & 1;
                    dim[m] = (p >> 1) + sec[m] * half;
                }
            }
#pragma unroll 1
            for (int row = 0; row < ANPD_ROWS; ++row) {
                float ss_row = 0.0f, best = -CUDART_INF_F;
                int bidx = 0x7fffffff;
                const float rstd = (EPI == RR_QKV || EPI == RR_GU || EPI == RR_LM) ? s_rstd[row] : 1.0f;
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    const int i = m * 128 + et, n = nn[m];
                    float y = 0.0f;
                    if (i < r) {
                        const float* col_tr = tr + (size_t)row * tr_stride + i;
                        for (int p = 0; p < P; ++p)                   // slices in ascending order, hi term then lo term
                            y += col_tr[(size_t)(p * 16) * tr_stride] + col_tr[(size_t)(p * 16 + ANPD_ROWS) * tr_stride];
                    }
                    if (!valid[m]) y = 0.0f;
                    if (EPI == RR_RAW) {
                        if (valid[m]) e.raw_out[(size_t)row * g.N + n] = y;
                    } else if (EPI == RR_QKV) {
                        const float mine0 = y * rstd;
                        const float other = __shfl_xor_sync(0xffffffffu, mine0, 1);
                        if (valid[m]) {
                            float mine = mine0;
                            if (head[m] < e.Hq + e.Hkv) {
                                const float cs = scratch[row * r + i], sn = scratch[ANPD_ROWS * r + row * r + i];
                                const float a = sec[m] ? other : mine0, b = sec[m] ? mine0 : other;      // (dimension i, dimension i + half)
                                mine = sec[m] ? (b * cs + a * sn) : (a * cs - b * sn);
                            }
                            if (head[m] < e.Hq) {
                                // queries leave as two bf16 terms, already multiplied by log2(e) / sqrt(hd)
                                const size_t o = (size_t)row * e.Hq * e.hd + (size_t)head[m] * e.hd + dim[m];
                                const float q = mine * e.q_scale;
                                const bf16 hi = __float2bfloat16_rn(q);
                                e.q_hi[o] = hi;
                                e.q_lo[o] = __float2bfloat16_rn(q - __bfloat162float(hi));
                            } else if (s_page[row] >= 0) {
                                const bool is_k = head[m] < e.Hq + e.Hkv;
                                const int kvh = is_k ? head[m] - e.Hq : head[m] - e.Hq - e.Hkv;
                                const int slot = s_pos[row] % KV_PAGE;
                                bf16* pg = (is_k ? e.kpool_l : e.vpool_l) + ((size_t)s_page[row] * e.Hkv + kvh) * KV_PAGE * e.hd;
                                if (is_k) pg[(size_t)slot * e.hd + dim[m]] = __float2bfloat16_rn(mine);     // K page: [position][dim]
                                else pg[(size_t)dim[m] * KV_PAGE + slot] = __float2bfloat16_rn(mine);       // V page: [dim][position]
                            }
                        }
                    } else if (EPI == RR_RESID) {
                        if (valid[m]) {
                            const float xn = scratch[row * r + i] + y;
                            e.x[(size_t)row * e.d + n] = xn;
                            split_store_row(e.act_out, col[m], row, xn * gn[m]);
                            ss_row += xn * xn;
                        }
                    } else if (EPI == RR_GU) {
                        const float mine = y * rstd;
                        const float other = __shfl_xor_sync(0xffffffffu, mine, 1);
                        if (valid[m] && !(n & 1)) split_store_row(e.act_out, col[m], row, mine / (1.0f + __expf(-mine)) * other);   // even feature: gate, odd neighbour: up
                    } else if (EPI == RR_LM) {
                        const float z = y * rstd;
                        if (valid[m] && n < e.V) {
                            if (e.logits) e.logits[(size_t)row * e.V + n] = z;
                            if (z > best) { best = z; bidx = n; }         // ascending n: strict > keeps the lowest id
                        }
                    }
                }
                // the row's reductions over the warp (fixed shuffle tree); the four warps are merged after the loop
                if (EPI == RR_RESID) {
                    for (int o = 16; o > 0; o >>= 1) ss_row += __shfl_xor_sync(0xffffffffu, ss_row, o);
                    if (lane == 0) red_f[ew][row] = ss_row;
                }
                if (EPI == RR_LM) {
                    for (int o = 16; o > 0; o >>= 1) {
                        const float ov = __shfl_xor_sync(0xffffffffu, best, o);
                        const int oi = __shfl_xor_sync(0xffffffffu, bidx, o);
                        if (ov > best || (ov == best && oi < bidx)) { best = ov; bidx = oi; }
                    }
                    if (lane == 0) { red_f[ew][row] = best; red_i[ew][row] = bidx; }
                }
            }
        } else if (lane == 0) {
#pragma unroll 1
            for (int row = 0; row < ANPD_ROWS; ++row) { red_f[ew][row] = EPI == RR_LM ? -CUDART_INF_F : 0.0f; red_i[ew][row] = 0x7fffffff; }
        }
        // CTA-wide part of the reductions: the four warps in warp order
        if (EPI == RR_RESID || EPI == RR_LM) {
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (ew == 0 && lane < ANPD_ROWS) {
                if (EPI == RR_RESID) {
                    e.ss_out[c * ANPD_ROWS + lane] = (red_f[0][lane] + red_f[1][lane]) + (red_f[2][lane] + red_f[3][lane]);
                } else {
                    float bv = red_f[0][lane];
                    int bi = red_i[0][lane];
                    for (int w = 1; w < 4; ++w)
                        if (red_f[w][lane] > bv || (red_f[w][lane] == bv && red_i[w][lane] < bi)) { bv = red_f[w][lane]; bi = red_i[w][lane]; }
                    e.amax_val[(size_t)lane * G + c] = bv;
                    e.amax_idx[(size_t)lane * G + c] = bi;
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)RR_TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && abort_flag) atomicExch(g.err, RR_ERR_TIMEOUT);
}

// Scatters rows [row_off, row_off + rows) of a row-major [rows][K] source into the row-range storage of the
// plan's matrix; `map` says where a source row goes among the (permuted) output features.
template <typename T>
__global__ void rr_retile_kernel(const T* __restrict__ src, int rows, int K, int row_off, int map, int hd, int F, RRPlanDev p,
                                 unsigned char* __restrict__ dst) {
    const int chunks = K / 8;                                  // 8 consecutive inputs = one 16-byte chunk of a 32-byte operand row
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < (size_t)rows * chunks; idx += (size_t)gridDim.x * blockDim.x) {
        const int rr = (int)(idx / chunks), k0 = (int)(idx % chunks) * 8;
        const int nf = row_off + rr;                           // row of the fused source matrix
        int n = nf;
        if (map == RR_MAP_HEADS) {                             // inside a head: dimension i -> 2i, dimension i + hd/2 -> 2i + 1
            const int head = nf / hd, dim = nf % hd, half = hd >> 1;
            n = head * hd + (dim % half) * 2 + dim / half;
        } else if (map == RR_MAP_GATE_UP) {                    // gate j -> 2j, up j -> 2j + 1
            n = nf < F ? 2 * nf : 2 * (nf - F) + 1;
        }
        const int pr = n >> 1;
        const int c = (int)((((long long)pr + 1) * p.G + p.pairs - 1) / p.pairs) - 1;        // owner: largest c with c * pairs / G <= pr
        const int first = 2 * (int)((long long)c * p.pairs / p.G);
        const int r = 2 * (int)((long long)(c + 1) * p.pairs / p.G) - first;                 // features of the owner
        const int f = n - first;
        const int ls = (k0 >> 6) / p.kb;                       // logical stage of this k-block
        int s = ls - (p.rotate ? rr_rotation(c, p.G, p.n_stages) : 0);                       // stored in the order the CTA reads
        if (s < 0) s += p.n_stages;
        const int q = (k0 >> 4) - ls * p.kb * 4;               // 16-wide slice within the stage
        const int t = q / p.P, sl = q % p.P;                   // step (instruction) and slice within it
        const int R = sl * r + f;                              // row of the step's N operand
        unsigned char* out = dst + ((unsigned long long)s * p.G + c) * p.slot_bytes + (size_t)t * p.w_step_global + (size_t)R * 32 +
                             (size_t)((((k0 >> 3) & 1) ^ ((R >> 2) & 1)) << 4);
        const T* in = src + (size_t)rr * K + k0;
        bf16 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = (bf16)in[u];
        *(uint4*)out = *(const uint4*)v;
    }
}

// fp32 activations [8][K] -> operand image (test hook)
__global__ void rr_act_image_kernel(const float* __restrict__ a, int K, unsigned char* __restrict__ img) {
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < ANPD_ROWS * K; idx += gridDim.x * blockDim.x)
        split_store(img, idx / K, idx % K, a[idx]);
}

template <int EPI, int MT>
anpd_status launch_rr_mt(const RRPlan& p, const RRArgs& g, const RREpi& e, cudaStream_t st, Profiler* prof) {
    static bool attr_set[64] = {false};
    if (first_call_on_device(attr_set)) {
        CUDA_TRY(cudaFuncSetAttribute(proj_rr_kernel<EPI, MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, 216 * 1024));
    }
    LAUNCH(prof, st, KC_GEMM, 2.0 * (double)p.N * (double)p.K,
           (launch_k(proj_rr_kernel<EPI, MT>, p.G, RR_THREADS, (size_t)p.smem_bytes, st, g, e)));
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}

template <int EPI>
anpd_status launch_rr(const RRPlan& p, const unsigned char* w, const unsigned char* act, const RREpi& e, int* err, cudaStream_t st, Profiler* prof) {
    RRArgs g;
    g.w = w; g.act = act; g.N = p.N; g.pairs = p.pairs; g.r_max = p.r_max; g.P = p.P; g.k_blocks = p.k_blocks; g.kb = p.kb;
    g.n_stages = p.n_stages; g.stages = p.stages; g.w_step_stride = p.w_step_stride; g.w_step_global = p.w_step_global; g.a_off = p.a_off;
    g.stage_bytes = p.stage_bytes; g.scratch_off = p.scratch_off; g.rotate = p.rotate; g.slot_bytes = p.slot_bytes; g.err = err;
    g.one_copy = (p.one_copy && p.w_step_stride == p.w_step_global) ? 1 : 0;
    return p.mt == 2 ? launch_rr_mt<EPI, 2>(p, g, e, st, prof) : launch_rr_mt<EPI, 1>(p, g, e, st, prof);
}

}  // namespace

void rr_make_plan(RRPlan* p, int N, int K, int num_sms) {
    p->N = N; p->K = K;
    p->pairs = (N + 1) / 2;
    p->G = std::min(num_sms, p->pairs);
    p->r_max = 2 * ((p->pairs + p->G - 1) / p->G);
    p->mt = (p->r_max + 127) / 128;                    // features per epilogue thread
    p->k_blocks = (K + 63) / 64;
    // slices per instruction: as many as fit 256 accumulator columns
    p->P = p->r_max * 8 <= 256 ? 8 : p->r_max * 4 <= 256 ? 4 : p->r_max * 2 <= 256 ? 2 : 1;
    p->w_step_global = p->P * p->r_max * 32;
    p->w_step_stride = (p->w_step_global + 255) & ~255;
    // k-blocks per stage: weight copies of about 16-24 KB per stage (whole instructions: two k-blocks each when P = 8)
    int kb = std::max(1, std::min(8, (int)((16384 + p->r_max * 64) / (p->r_max * 128))));
    if (const char* s = std::getenv("ANPD_RR_KB")) kb = std::max(1, std::min(8, std::atoi(s)));
    if (p->P == 8) kb = std::max(2, kb & ~1);
    while (kb > 1 && (kb * 4 + p->P - 1) / p->P > RR_MAX_STEPS) kb -= (p->P == 8 ? 2 : 1);      // the MMA issuer unrolls this many steps
    kb = std::min(kb, std::max(1, p->k_blocks));
    if (p->P == 8) kb = std::max(2, (kb + 1) & ~1);
    p->kb = kb;
    p->n_stages = (p->k_blocks + kb - 1) / kb;
    const int sps = (kb * 4 + p->P - 1) / p->P;        // steps per stage
    p->a_off = sps * p->w_step_stride;
    p->stage_bytes = p->a_off + kb * A_KB_BYTES;
    // An instruction reads 128 operand rows of activations (4 KB) and up to 15 rows of weights more than are real: the
    // last step of the ring's last stage reads past the stage.  Keep that inside the allocation.
    const int over_read = 4096 + 512;
    int budget = 107 * 1024;               // two such CTAs fit one SM: the next projection fills its ring while this one streams
    if (const char* s = std::getenv("ANPD_RR_RING_KB")) budget = std::max(32, std::min(180, std::atoi(s))) * 1024;
    const int scratch = 2 * ANPD_ROWS * p->r_max * 4;      // per (row, feature): two rotary factors, or one residual value
    p->stages = std::max(2, std::min(RR_MAX_STAGES, (budget - over_read - scratch - 1024) / p->stage_bytes));
    p->rotate = std::getenv("ANPD_RR_NO_ROTATE") == nullptr ? 1 : 0;
    p->one_copy = std::getenv("ANPD_RR_ONE_COPY") != nullptr ? 1 : 0;
    p->slot_bytes = (unsigned long long)sps * p->w_step_global;
    p->scratch_off = p->stages * p->stage_bytes + over_read;
    p->smem_bytes = p->scratch_off + scratch + 1024;
}

size_t rr_storage_bytes(const RRPlan& p) { return (size_t)p.n_stages * p.G * p.slot_bytes; }

anpd_status rr_retile_enqueue(const RRPlan& p, const void* src, bool src_is_f32, int rows, int row_off, int map, int hd, int F,
                              unsigned char* dst, cudaStream_t st) {
    RRPlanDev d{p.G, p.pairs, p.r_max, p.kb, p.n_stages, p.rotate, p.P, p.w_step_global, p.slot_bytes};
    const size_t work = (size_t)rows * (p.K / 8);
    const int blocks = (int)std::min<size_t>((work + 255) / 256, 148 * 16);
    if (src_is_f32) rr_retile_kernel<float><<<blocks, 256, 0, st>>>((const float*)src, rows, p.K, row_off, map, hd, F, d, dst);
    else rr_retile_kernel<bf16><<<blocks, 256, 0, st>>>((const bf16*)src, rows, p.K, row_off, map, hd, F, d, dst);
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}

anpd_status rr_act_image_enqueue(const float* a_dev, int K, unsigned char* img, cudaStream_t st) {
    rr_act_image_kernel<<<32, 256, 0, st>>>(a_dev, K, img);
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}

anpd_status rr_enqueue(int epi, const RRPlan& p, const unsigned char* w, const unsigned char* act, const RREpiHost& h, int* err,
                       cudaStream_t st, Profiler* prof) {
    RREpi e;
    e.ss_in = h.ss_in; e.n_parts_in = h.n_parts_in; e.inv_d_in = h.inv_d_in; e.eps = h.eps;
    e.row_pos = h.row_pos; e.row_seq = h.row_seq; e.row_ok = h.row_ok; e.rope_cos = h.rope_cos; e.rope_sin = h.rope_sin;
    e.page_table = h.page_table; e.pages_per_seq = h.pages_per_seq; e.Hq = h.Hq; e.Hkv = h.Hkv; e.hd = h.hd; e.q_scale = h.q_scale;
    e.q_hi = h.q_hi; e.q_lo = h.q_lo; e.kpool_l = h.kpool_l; e.vpool_l = h.vpool_l;
    e.x = h.x; e.gain = h.gain; e.ss_out = h.ss_out; e.d = h.d; e.act_out = h.act_out;
    e.logits = h.logits; e.amax_val = h.amax_val; e.amax_idx = h.amax_idx; e.V = h.V; e.raw_out = h.raw_out;
    switch (epi) {
        case RR_RAW: return launch_rr<RR_RAW>(p, w, act, e, err, st, prof);
        case RR_QKV: return launch_rr<RR_QKV>(p, w, act, e, err, st, prof);
        case RR_RESID: return launch_rr<RR_RESID>(p, w, act, e, err, st, prof);
        case RR_GU: return launch_rr<RR_GU>(p, w, act, e, err, st, prof);
        case RR_LM: return launch_rr<RR_LM>(p, w, act, e, err, st, prof);
    }
    return ANPD_ERR_ARG;
}
