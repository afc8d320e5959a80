// anpd_gemm_static: the weight-streaming GEMM for callers that must not allocate.
//
// Some users of this library cannot let it call cudaMalloc: a serving loop in which the implicit
// device-wide synchronisation of an allocation would stall every other stream, or a process whose
// whole device memory has already been handed to another allocator (a framework's memory pool), so
// that an allocation made behind its back may simply fail.  anpd_debug_gemm allocates its weight
// staging, activation and partial-sum buffers on every call; this variant computes the same product
// with all of that scratch in one fixed array that is part of the loaded library image.
//
// The scratch array is shared by every call on a device and keeps whatever the last call left in
// it.  The call clears what has to start at zero (the padded weight blocks and the error flag) and
// overwrites the rest before reading it.  Two calls that overlap on the GPU (different streams, or
// different host threads) would use the same scratch at once and corrupt each other: run them one
// after the other.
#include "internal.h"

#include <cstdio>

typedef __nv_bfloat16 bf16;

namespace {

constexpr int MAX_BLOCKS = 128;                     // ceil(N/128) * ceil(K/64) accepted by the entry point
constexpr int MAX_SLOTS = 256;                      // block slots held (the block order pads up to a multiple of the grid)
constexpr int MAX_ROWS = 32;
constexpr size_t W_BYTES = (size_t)MAX_SLOTS * 128 * 64 * 2;                 // 4 MiB   weight blocks
constexpr size_t A_BYTES_EACH = (size_t)MAX_ROWS * MAX_BLOCKS * 64 * 2;      // 512 KiB one bf16 term of the activations
constexpr size_t P_BYTES = (size_t)MAX_BLOCKS * 128 * MAX_ROWS * 4;          // 2 MiB   partial sums
constexpr size_t T_BYTES = 2 * 1024;                                         // per-tile tables
constexpr size_t E_BYTES = 256;                                              // error flag
constexpr size_t OFF_HI = W_BYTES, OFF_LO = OFF_HI + A_BYTES_EACH, OFF_PART = OFF_LO + A_BYTES_EACH,
                 OFF_FIRST = OFF_PART + P_BYTES, OFF_SEGS = OFF_FIRST + T_BYTES / 2, OFF_ERR = OFF_FIRST + T_BYTES,
                 SCRATCH_BYTES = OFF_ERR + E_BYTES;                          // about 7 MiB in all

// Lives in every GPU's memory from the moment the library is loaded there until the process ends.
// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[SCRATCH_BYTES];

// Device address of the scratch array per device ordinal, looked up once per device.
constexpr int MAX_DEVICES = 64;
void* g_scratch_addr[MAX_DEVICES] = {nullptr};

// Which CTA starts each tile and how many CTAs (= partial sums) cover it, for the equal split of
// the (tile, k-block) sequence over G CTAs.
__global__ void static_plan_kernel(int* first_cta, int* seg_count, int m_tiles, int k_blocks, long long total, int G) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= m_tiles) return;
    const long long b0 = (long long)t * k_blocks, b1 = b0 + k_blocks - 1;
    const int c0 = (int)(((b0 + 1) * G + total - 1) / total - 1), c1 = (int)(((b1 + 1) * G + total - 1) / total - 1);
    first_cta[t] = c0;
    seg_count[t] = c1 - c0 + 1;
}

// fp32 activations -> two bf16 terms (hi = nearest bf16, lo = nearest bf16 of the remainder).
__global__ void static_split_kernel(const float* __restrict__ a, bf16* __restrict__ hi, bf16* __restrict__ lo, size_t n) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const float v = a[i];
        const bf16 h = __float2bfloat16_rn(v);
        hi[i] = h;
        lo[i] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
}

// out[row][n] = the tile's partial sums added in segment (ascending K) order.
__global__ void static_reduce_kernel(const float* __restrict__ part, const int* __restrict__ seg_count, int rows, int N,
                                     float* __restrict__ out) {
    const size_t total = (size_t)rows * N;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int n = (int)(i % N);
        const int ns = seg_count[n >> 7];
        float acc = 0.0f;
        for (int s = 0; s < ns; ++s) acc += part[(size_t)s * total + i];
        out[i] = acc;
    }
}

}  // namespace

extern "C" anpd_status anpd_gemm_static(const uint16_t* w_bf16_dev, int N, int K, const float* a_dev, int rows,
                                        float* out_dev, void* cuda_stream) {
    if (!w_bf16_dev || !a_dev || !out_dev || N < 1 || K < 8 || K % 8 || rows < 8 || rows % 8) return ANPD_ERR_ARG;
    const int m_tiles = (N + 127) / 128, k_blocks = (K + 63) / 64;
    const long long total = (long long)m_tiles * k_blocks;
    if (rows > MAX_ROWS || total > MAX_BLOCKS) {
        std::fprintf(stderr, "[anpd] anpd_gemm_static: %d rows and %lld weight blocks (ceil(N/128) * ceil(K/64)) exceed the fixed "
                             "scratch: at most %d rows and %d blocks\n", rows, total, MAX_ROWS, MAX_BLOCKS);
        return ANPD_ERR_CAPACITY;
    }
    int dev = 0, sms = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return ANPD_ERR_ARG;
    if (!g_scratch_addr[dev]) {
        // one-time set-up for this device: the device address behind the symbol
        void* p = nullptr;
        CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
        g_scratch_addr[dev] = p;
    }
    unsigned char* scratch = (unsigned char*)g_scratch_addr[dev];
    CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));

    // the scalar part of the GEMM plan (the per-tile tables are computed on the device)
    GemmPlan plan;
    plan.N = N; plan.K = K; plan.m_tiles = m_tiles; plan.k_blocks = k_blocks;
    plan.grid = (int)(total < sms ? total : sms);
    plan.max_count = (int)((total + plan.grid - 1) / plan.grid);
    plan.max_segs = 0;
    plan.d_first_cta = (int*)(scratch + OFF_FIRST);
    plan.d_seg_count = (int*)(scratch + OFF_SEGS);
    if ((long long)plan.max_count * plan.grid > MAX_SLOTS) return ANPD_ERR_CAPACITY;

    cudaStream_t st = (cudaStream_t)cuda_stream;
    bf16* d_w = (bf16*)scratch;
    bf16* d_hi = (bf16*)(scratch + OFF_HI);
    bf16* d_lo = (bf16*)(scratch + OFF_LO);
    float* d_part = (float*)(scratch + OFF_PART);
    int* d_err = (int*)(scratch + OFF_ERR);
    const int NB = (rows + 15) / 16 * 16;

    // stale contents of the last call: the weight blocks' padding and the error flag must be zero
    CUDA_TRY(cudaMemsetAsync(d_w, 0, gemm_tiled_elems(plan) * 2, st));
    CUDA_TRY(cudaMemsetAsync(d_err, 0, sizeof(int), st));
    static_plan_kernel<<<1, 128, 0, st>>>(plan.d_first_cta, plan.d_seg_count, m_tiles, k_blocks, total, plan.grid);
    static_split_kernel<<<64, 256, 0, st>>>(a_dev, d_hi, d_lo, (size_t)rows * K);
    CUDA_TRY(cudaGetLastError());
    ANPD_TRY(gemm_retile_enqueue(plan, w_bf16_dev, false, N, 0, d_w, st));
    CUtensorMap mh, ml;
    ANPD_TRY(make_tmap_bf16(&mh, d_hi, rows, K, NB, false));
    ANPD_TRY(make_tmap_bf16(&ml, d_lo, rows, K, NB, false));
    {
        // The GEMM kernel requests its first weight blocks ahead of its dependency wait, which is only sound for
        // weights no earlier kernel of the stream writes.  Here the blocks were written by the kernels just above,
        // so this launch must not overlap them: no programmatic dependent launch.
        NoPdlScope ordered(true);
        ANPD_TRY(gemm_tc_enqueue(plan, d_w, mh, ml, rows, NB, d_part, (size_t)rows * N, N, d_err, st, nullptr));
    }
    static_reduce_kernel<<<64, 256, 0, st>>>(d_part, plan.d_seg_count, rows, N, out_dev);
    CUDA_TRY(cudaGetLastError());
    int err = 0;
    CUDA_TRY(cudaMemcpyAsync(&err, d_err, sizeof(int), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    return err == 0 ? ANPD_OK : ANPD_ERR_CUDA;
}
