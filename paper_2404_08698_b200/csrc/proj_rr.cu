// Projections of a single-sequence verify step (8 rows) with everything that follows them fused in:
//   QKV     -> rotary embedding, query scaling, K/V rows appended to the paged cache
//   O, down -> residual add, the next RMSNorm's gain, the row's sum of squares (partial)
//   gate/up -> SwiGLU
//   LM head -> logits (optional) and the per-CTA argmax
// (paper Section 3.1, "Verification": the forward over the K+1 tokens of a step.)
//
// The step is bound by reading every weight once.  Here each of the G = #SMs CTAs owns a contiguous
// range of OUTPUT FEATURES of the matrix (about N / G weight rows) and walks the whole contraction
// dimension, so a CTA ends with complete dot products and can finish the layer's elementwise work in
// its epilogue: no partial sums cross CTAs, and the small kernels that used to sit between two
// projections (each a dependent launch with its own memory round trip) are gone.
//
//   - operands swapped as in the stream-K kernel: the CTA's r weight rows are the MMA's M operand
//     (M = 128 per instruction; rows beyond r read whatever follows in shared memory and produce
//     accumulator lanes nobody reads), the step's 8 rows are the N operand, as hi terms (rows 0-7)
//     and lo terms (rows 8-15) of one 16-row tile: N = 16, one accumulator of 16 columns per M tile;
//   - the weights are stored, per CTA, as the exact shared-memory image of its k-blocks (r rows of
//     128 bytes, 128-byte swizzle), stage after stage, stages of all CTAs side by side: at any time
//     the G CTAs read one contiguous window that sweeps through memory; r need not be a multiple of
//     8, so the ranges differ by at most one feature pair and every SM streams the same bytes;
//   - the activations arrive as a ready-made operand image too (written by the producing epilogue),
//     2 KB per k-block, fetched by one linear bulk copy per stage;
//   - RMSNorm is deferred: the producer of the residual stream writes x * gain (hi + lo) and each
//     CTA's partial sum of squares; the consuming projection multiplies its outputs by
//     1 / rms(x), which commutes with the matrix product.  Partial sums are added in CTA order,
//     so the result is the same bits in every launch.
// Features are permuted at model creation so that the two members of a rotary pair (dimension i and
// i + head_dim/2) and of a SwiGLU pair (gate j, up j) are neighbours; a CTA's range starts at an even
// feature, so a pair never straddles CTAs, warps or M tiles and is exchanged with one shuffle.
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
constexpr int B_TILE_BYTES = 16 * 128;   // one k-block of the activation operand: 8 hi rows + 8 lo rows x 64 bf16

struct RRArgs {
    const unsigned char* w;              // this matrix in row-range storage
    const unsigned char* act;            // activation operand image, B_TILE_BYTES per k-block
    int N;                               // output features (valid)
    int pairs;                           // feature pairs = ceil(N / 2), cut evenly across the grid
    int r_max;                           // most features a CTA owns
    int k_blocks, kb, n_stages, stages;
    int a_tile_stride;                   // bytes between the weight tiles of two k-blocks inside a stage
    int stage_bytes;
    int mt;                              // 128-row M tiles per CTA (1 or 2)
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

template <int EPI>
__global__ void __launch_bounds__(RR_THREADS, 1) proj_rr_kernel(const RRArgs g, const RREpi e) {
    extern __shared__ __align__(1024) unsigned char rr_smem_raw[];
    __shared__ uint64_t bar_full[RR_MAX_STAGES], bar_empty[RR_MAX_STAGES], bar_done;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ float red_f[4][ANPD_ROWS];
    __shared__ int red_i[4][ANPD_ROWS];

    pdl_trigger();
    unsigned char* smem = rr_smem_raw + ((1024u - (smem_u32(rr_smem_raw) & 1023u)) & 1023u);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, c = blockIdx.x;
    const int start = 2 * (int)((long long)c * g.pairs / G);
    const int r = 2 * (int)((long long)(c + 1) * g.pairs / G) - start;          // features of this CTA
    const int a_bytes = g.kb * g.a_tile_stride;                                  // weight part of a stage

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < g.stages; ++s) { mbar_init(&bar_full[s], 1); mbar_init(&bar_empty[s], 1); }
        mbar_init(&bar_done, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(32u) : "memory");
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
            const uint32_t w_row_bytes = (uint32_t)r * 128u;
            auto kbs = [&](int s) { return min(g.kb, g.k_blocks - s * g.kb); };
            auto load_w = [&](int s, int stage) {
                const int n = kbs(s);
                mbar_expect_tx(&bar_full[stage], (uint32_t)n * (w_row_bytes + B_TILE_BYTES));
                const unsigned char* src = g.w + ((unsigned long long)s * G + c) * g.slot_bytes;
                unsigned char* dst = smem + (size_t)stage * g.stage_bytes;
                for (int j = 0; j < n; ++j)
                    bulk_load(dst + (size_t)j * g.a_tile_stride, src + (size_t)j * g.r_max * 128, w_row_bytes, &bar_full[stage], pol_w);
            };
            auto load_b = [&](int s, int stage) {
                bulk_load(smem + (size_t)stage * g.stage_bytes + a_bytes, g.act + (size_t)s * g.kb * B_TILE_BYTES,
                          (uint32_t)kbs(s) * B_TILE_BYTES, &bar_full[stage], pol_a);
            };
            // the weights depend on no earlier kernel: fill the ring first, then wait for the activations' producer
            const int ahead = min(g.stages, g.n_stages);
            for (int s = 0; s < ahead; ++s) load_w(s, s);
            pdl_wait();
            for (int s = 0; s < ahead; ++s) load_b(s, s);
            int stage = ahead % g.stages;
            uint32_t phase = (ahead == g.stages) ? 1u : 0u;
            int issued = ahead;
            bool ok = true;
            for (int s = ahead; s < g.n_stages; ++s) {
                ok = mbar_wait(&bar_empty[stage], phase ^ 1u, abortp);
                if (!ok) break;
                load_w(s, stage);
                load_b(s, stage);
                ++issued;
                if (++stage == g.stages) { stage = 0; phase ^= 1u; }
            }
            if (!ok) {
                // gave up: let every copy already issued land before the CTA may exit
                const int n = issued < g.stages ? issued : g.stages;
                for (int i = 0; i < n; ++i) {
                    const int idx = issued - 1 - i;
                    const int s = idx % g.stages;
                    const uint32_t ph = (uint32_t)((idx / g.stages) & 1);
                    for (unsigned spin = 0; spin < WAIT_LIMIT && !mbar_try_wait(&bar_full[s], ph); ++spin) {}
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            // fp32 accumulate, bf16 x bf16, both operands K-major, M = 128, N = 16
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(16 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            uint32_t acc = 0;
            for (int s = 0; s < g.n_stages && ok; ++s) {
                ok = mbar_wait(&bar_full[stage], phase, abortp);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sa = smem_u32(smem + (size_t)stage * g.stage_bytes);
                const int n = min(g.kb, g.k_blocks - s * g.kb);
                for (int j = 0; j < n; ++j) {
                    const uint64_t db = make_smem_desc(sa + a_bytes + j * B_TILE_BYTES);
#pragma unroll
                    for (int k16 = 0; k16 < 4; ++k16) {
                        const uint64_t adv = (uint64_t)(k16 * 2);           // 16 bf16 = 32 bytes along K inside the swizzle row
                        for (int m = 0; m < g.mt; ++m)
                            tc_mma_bf16(tmem_base + (uint32_t)(m * 16), make_smem_desc(sa + j * g.a_tile_stride + m * 16384) + adv, db + adv, idesc, acc);
                        acc = 1;
                    }
                }
                tc_commit(&bar_empty[stage]);            // frees the stage once these MMAs have read it
                if (++stage == g.stages) { stage = 0; phase ^= 1u; }
            }
            if (ok) tc_commit(&bar_done);
        }
    } else {
        // ---------------- epilogue warps ----------------
        const int quad = warp & 3;                        // a warp may only touch TMEM lanes 32 * (warp % 4) .. + 31
        const int ew = warp - 2;                          // 0..3
        pdl_wait();
        // work that needs no accumulator, done while the weights stream
        float rstd[ANPD_ROWS];
        if (EPI == RR_QKV || EPI == RR_GU || EPI == RR_LM) {
#pragma unroll
            for (int row = 0; row < ANPD_ROWS; ++row) {
                float s = 0.0f;
                for (int i = lane; i < e.n_parts_in; i += 32) s += e.ss_in[i * ANPD_ROWS + row];
                for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                rstd[row] = rsqrtf(s * e.inv_d_in + e.eps);
            }
        }
        float xin[2][ANPD_ROWS], gn[2] = {0.f, 0.f};
        if (EPI == RR_RESID) {
            for (int m = 0; m < g.mt; ++m) {
                const int i = m * 128 + quad * 32 + lane, n = start + i;
                const bool valid = i < r && n < g.N;
                gn[m] = valid ? e.gain[n] : 0.0f;
#pragma unroll
                for (int row = 0; row < ANPD_ROWS; ++row) xin[m][row] = valid ? e.x[(size_t)row * e.d + n] : 0.0f;
            }
        }
        int pos[ANPD_ROWS];
        if (EPI == RR_QKV) {
#pragma unroll
            for (int row = 0; row < ANPD_ROWS; ++row) pos[row] = e.row_pos[row];
        }
        const bool ok = mbar_wait(&bar_done, 0, abortp);
        tc_fence_after();
        float ss[ANPD_ROWS];
        float best[ANPD_ROWS];
        int bidx[ANPD_ROWS];
#pragma unroll
        for (int row = 0; row < ANPD_ROWS; ++row) { ss[row] = 0.0f; best[row] = -CUDART_INF_F; bidx[row] = 0x7fffffff; }
        if (ok) {
            for (int m = 0; m < g.mt; ++m) {
                const int i = m * 128 + quad * 32 + lane, n = start + i;
                const bool valid = i < r && n < g.N;
                float v[16], y[ANPD_ROWS];
                tc_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(m * 16), v);
#pragma unroll
                for (int row = 0; row < ANPD_ROWS; ++row) y[row] = valid ? v[row] + v[ANPD_ROWS + row] : 0.0f;
                if (EPI == RR_RAW) {
                    if (valid)
#pragma unroll
                        for (int row = 0; row < ANPD_ROWS; ++row) e.raw_out[(size_t)row * g.N + n] = y[row];
                } else if (EPI == RR_QKV) {
                    const int half = e.hd >> 1;
                    const int head = n / e.hd, p = n - head * e.hd, sec = p & 1, dim = (p >> 1) + sec * half;
#pragma unroll
                    for (int row = 0; row < ANPD_ROWS; ++row) {
                        const float mine0 = y[row] * rstd[row];
                        const float other = __shfl_xor_sync(0xffffffffu, mine0, 1);
                        if (!valid) continue;
                        float mine = mine0;
                        if (head < e.Hq + e.Hkv) {
                            const float cs = e.rope_cos[(size_t)pos[row] * half + (p >> 1)], sn = e.rope_sin[(size_t)pos[row] * half + (p >> 1)];
                            const float a = sec ? other : mine0, b = sec ? mine0 : other;      // (dimension i, dimension i + half)
                            mine = sec ? (b * cs + a * sn) : (a * cs - b * sn);
                        }
                        if (head < e.Hq) {
                            // queries leave as two bf16 terms, already multiplied by log2(e) / sqrt(hd)
                            const size_t o = (size_t)row * e.Hq * e.hd + (size_t)head * e.hd + dim;
                            const float q = mine * e.q_scale;
                            const bf16 hi = __float2bfloat16_rn(q);
                            e.q_hi[o] = hi;
                            e.q_lo[o] = __float2bfloat16_rn(q - __bfloat162float(hi));
                        } else if (e.row_ok[row]) {
                            const bool is_k = head < e.Hq + e.Hkv;
                            const int kvh = is_k ? head - e.Hq : head - e.Hq - e.Hkv;
                            const int page = e.page_table[e.row_seq[row] * e.pages_per_seq + pos[row] / KV_PAGE];
                            bf16* pg = (is_k ? e.kpool_l : e.vpool_l) + ((size_t)page * e.Hkv + kvh) * KV_PAGE * e.hd;
                            if (is_k) pg[(size_t)(pos[row] % KV_PAGE) * e.hd + dim] = __float2bfloat16_rn(mine);     // K page: [position][dim]
                            else pg[(size_t)dim * KV_PAGE + (pos[row] % KV_PAGE)] = __float2bfloat16_rn(mine);       // V page: [dim][position]
                        }
                    }
                } else if (EPI == RR_RESID) {
#pragma unroll
                    for (int row = 0; row < ANPD_ROWS; ++row) {
                        const float xn = xin[m][row] + y[row];
                        if (valid) {
                            e.x[(size_t)row * e.d + n] = xn;
                            split_store(e.act_out, row, n, xn * gn[m]);
                            ss[row] += xn * xn;
                        }
                    }
                } else if (EPI == RR_GU) {
#pragma unroll
                    for (int row = 0; row < ANPD_ROWS; ++row) {
                        const float mine = y[row] * rstd[row];
                        const float other = __shfl_xor_sync(0xffffffffu, mine, 1);
                        if (valid && !(n & 1)) split_store(e.act_out, row, n >> 1, mine / (1.0f + expf(-mine)) * other);   // even: gate, odd: up
                    }
                } else if (EPI == RR_LM) {
                    const bool real = valid && n < e.V;
#pragma unroll
                    for (int row = 0; row < ANPD_ROWS; ++row) {
                        const float z = y[row] * rstd[row];
                        if (real) {
                            if (e.logits) e.logits[(size_t)row * e.V + n] = z;
                            if (z > best[row]) { best[row] = z; bidx[row] = n; }      // ascending n: strict > keeps the lowest id
                        }
                    }
                }
            }
        }
        tc_fence_before();
        // CTA-wide reductions of the epilogue (fixed order: lanes by shuffle tree, then the four warps in order)
        if (EPI == RR_RESID) {
#pragma unroll
            for (int row = 0; row < ANPD_ROWS; ++row) {
                float s = ss[row];
                for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                if (lane == 0) red_f[ew][row] = s;
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (ew == 0 && lane < ANPD_ROWS)
                e.ss_out[c * ANPD_ROWS + lane] = (red_f[0][lane] + red_f[1][lane]) + (red_f[2][lane] + red_f[3][lane]);
        }
        if (EPI == RR_LM) {
#pragma unroll
            for (int row = 0; row < ANPD_ROWS; ++row) {
                float bv = best[row];
                int bi = bidx[row];
                for (int o = 16; o > 0; o >>= 1) {
                    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                    if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
                }
                if (lane == 0) { red_f[ew][row] = bv; red_i[ew][row] = bi; }
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (ew == 0 && lane < ANPD_ROWS) {
                float bv = red_f[0][lane];
                int bi = red_i[0][lane];
                for (int w = 1; w < 4; ++w)
                    if (red_f[w][lane] > bv || (red_f[w][lane] == bv && red_i[w][lane] < bi)) { bv = red_f[w][lane]; bi = red_i[w][lane]; }
                e.amax_val[(size_t)lane * G + c] = bv;
                e.amax_idx[(size_t)lane * G + c] = bi;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(32u) : "memory");
    }
    if (threadIdx.x == 0 && abort_flag) atomicExch(g.err, RR_ERR_TIMEOUT);
}

// Scatters rows [row_off, row_off + rows) of a row-major [rows][K] source into the row-range storage of the
// plan's matrix; `map` says where a source row goes among the (permuted) output features.
template <typename T>
__global__ void rr_retile_kernel(const T* __restrict__ src, int rows, int K, int row_off, int map, int hd, int F, RRPlanDev p,
                                 unsigned char* __restrict__ dst) {
    const int chunks = K / 8;                                  // 8 consecutive inputs never straddle a 64-wide k-block
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
        const int i = n - 2 * (int)((long long)c * p.pairs / p.G);
        const int kblk = k0 >> 6, s = kblk / p.kb, j = kblk % p.kb, kk = k0 & 63;
        unsigned char* out = dst + ((unsigned long long)s * p.G + c) * p.slot_bytes + (size_t)j * p.r_max * 128 + (size_t)i * 128 +
                             (size_t)(((kk >> 3) ^ (i & 7)) << 4);
        const T* in = src + (size_t)rr * K + k0;
        bf16 v[8];
#pragma unroll
        for (int t = 0; t < 8; ++t) v[t] = (bf16)in[t];
        *(uint4*)out = *(const uint4*)v;
    }
}

// fp32 activations [8][K] -> operand image (test hook)
__global__ void rr_act_image_kernel(const float* __restrict__ a, int K, unsigned char* __restrict__ img) {
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < ANPD_ROWS * K; idx += gridDim.x * blockDim.x)
        split_store(img, idx / K, idx % K, a[idx]);
}

template <int EPI>
anpd_status launch_rr(const RRPlan& p, const unsigned char* w, const unsigned char* act, const RREpi& e, int* err, cudaStream_t st, Profiler* prof) {
    static bool attr_set[64] = {false};
    if (first_call_on_device(attr_set)) {
        CUDA_TRY(cudaFuncSetAttribute(proj_rr_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, 216 * 1024));
    }
    RRArgs g;
    g.w = w; g.act = act; g.N = p.N; g.pairs = p.pairs; g.r_max = p.r_max; g.k_blocks = p.k_blocks; g.kb = p.kb;
    g.n_stages = p.n_stages; g.stages = p.stages; g.a_tile_stride = p.a_tile_stride; g.stage_bytes = p.stage_bytes; g.mt = p.mt;
    g.slot_bytes = p.slot_bytes; g.err = err;
    LAUNCH(prof, st, KC_GEMM, 2.0 * (double)p.N * (double)p.K,
           (launch_k(proj_rr_kernel<EPI>, p.G, RR_THREADS, (size_t)p.smem_bytes, st, g, e)));
    CUDA_TRY(cudaGetLastError());
    return ANPD_OK;
}

}  // namespace

void rr_make_plan(RRPlan* p, int N, int K, int num_sms) {
    p->N = N; p->K = K;
    p->pairs = (N + 1) / 2;
    p->G = std::min(num_sms, p->pairs);
    p->r_max = 2 * ((p->pairs + p->G - 1) / p->G);
    p->mt = (p->r_max + 127) / 128;
    p->k_blocks = (K + 63) / 64;
    p->a_tile_stride = (p->r_max + 7) / 8 * 1024;
    // k-blocks per stage: copies of about 16 KB; ring: about 100 KB per CTA, so that the next projection's CTA fits
    // beside this one and fills its own ring while this one is still streaming
    int kb = std::max(1, std::min(8, (int)((16384 + p->r_max * 64) / (p->r_max * 128))));
    if (const char* s = std::getenv("ANPD_RR_KB")) kb = std::max(1, std::min(8, std::atoi(s)));
    kb = std::min(kb, p->k_blocks);
    p->kb = kb;
    p->n_stages = (p->k_blocks + kb - 1) / kb;
    p->stage_bytes = kb * (p->a_tile_stride + B_TILE_BYTES);
    // An MMA always reads 128 rows per M tile: the last tile of a stage's last k-block reads past its own rows, over
    // the stage's activation tiles and beyond.  Keep that inside the allocation.
    const int over_read = std::max(0, 128 * p->mt * 128 - p->a_tile_stride - kb * B_TILE_BYTES);
    int budget = 107 * 1024;               // two such CTAs fit one SM
    if (const char* s = std::getenv("ANPD_RR_RING_KB")) budget = std::max(32, std::min(180, std::atoi(s))) * 1024;
    p->stages = std::max(2, std::min(RR_MAX_STAGES, (budget - over_read - 1024) / p->stage_bytes));
    p->slot_bytes = (unsigned long long)kb * p->r_max * 128;
    p->smem_bytes = p->stages * p->stage_bytes + over_read + 1024;
}

size_t rr_storage_bytes(const RRPlan& p) { return (size_t)p.n_stages * p.G * p.slot_bytes; }

anpd_status rr_retile_enqueue(const RRPlan& p, const void* src, bool src_is_f32, int rows, int row_off, int map, int hd, int F,
                              unsigned char* dst, cudaStream_t st) {
    RRPlanDev d{p.G, p.pairs, p.r_max, p.kb, p.slot_bytes};
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
