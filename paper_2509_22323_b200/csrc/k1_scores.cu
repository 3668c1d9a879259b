// K1: pooled block scores.
//   pool_kernel   : one warp per (Q|K, image, head, 64-token block); 128-bit coalesced loads,
//                   fp64 accumulation, mean over the valid tokens of the block.
//                   HBM-bound: reads Q and K exactly once.
//   scores_kernel : S[i][j] = Qbar[i,:] . Kbar[j,:] in fp64 (fp64 mma.sync fragments), rounded once to fp32.
#include "common.cuh"

namespace {

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// One warp per (Q|K, image, head, 64-token block).  A token row of D channels is D / 8 lanes of
// 16 bytes, so one warp-wide load covers 32 / (D / 8) rows; every lane keeps fp64 sums of its 8
// channels over the rows it sees (eight loads in flight per lane), and the lanes that hold the
// same channels are then added with shuffles.  No shared memory.  The batches of eight loads are not unrolled into
// one another: that keeps the kernel under 85 registers, six thread blocks per SM (measured 29 against 40 us on the
// FLUX 1024^2 shapes, where 125 registers left four).
template <int D>
__global__ void __launch_bounds__(128, 6) pool_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k,
                                                   TensorGeom g, ImgList imgs, double* __restrict__ pooled,
                                                   const DevPlan* __restrict__ plan, int n_cap) {
    constexpr int TPR = D / 8;          // lanes per token row (8 channels = 16 bytes each)
    constexpr int RPL = 32 / TPR;       // rows per warp-wide load
    constexpr int ITERS = 64 / RPL;     // loads per lane
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int blk = blockIdx.x * 4 + warp, h = blockIdx.y;
    grid_dependency_launch();                         // the scores kernel may be staged; it waits for this grid's end itself
    if (blk >= g.nb) return;
    const int which = blockIdx.z / n_cap;             // 0 = Q, 1 = K
    const int p = blockIdx.z - which * n_cap;
    if (plan && p >= plan->sparse.n) return;          // device-resident plan: fewer images than the grid covers
    const int batch = plan ? plan->sparse.batch[p] : imgs.batch[p];
    const uint16_t* base = (which ? k : q) + (long long)batch * g.stride_b + (long long)(g.h0 + h) * g.stride_h;
    const int c = lane % TPR, r0 = lane / TPR;
    const int n0 = blk * 64;
    const int valid = min(64, g.N - n0);

    double acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.0;
#pragma unroll 1
    for (int it0 = 0; it0 < ITERS; it0 += 8) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int row = (it0 + u) * RPL + r0;
            v[u] = make_uint4(0, 0, 0, 0);
            if (row < valid)
                v[u] = __ldg(reinterpret_cast<const uint4*>(base + (long long)(n0 + row) * g.stride_n + c * 8));
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            acc[0] += (double)bf16_lo(v[u].x); acc[1] += (double)bf16_hi(v[u].x);
            acc[2] += (double)bf16_lo(v[u].y); acc[3] += (double)bf16_hi(v[u].y);
            acc[4] += (double)bf16_lo(v[u].z); acc[5] += (double)bf16_hi(v[u].z);
            acc[6] += (double)bf16_lo(v[u].w); acc[7] += (double)bf16_hi(v[u].w);
        }
    }
#pragma unroll
    for (int off = TPR; off < 32; off <<= 1)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], off);
    if (lane < TPR) {
        double* o = pooled + ((((long long)which * n_cap + p) * g.H + h) * g.nb + blk) * D + c * 8;
        const double inv = 1.0 / (double)valid;
#pragma unroll
        for (int e = 0; e < 8; e += 2) {
            double2 w2 = make_double2(acc[e] * inv, acc[e + 1] * inv);
            *reinterpret_cast<double2*>(o + e) = w2;
        }
    }
}

// D(8 x 8, fp64) += A(8 x 4, row) * B(4 x 8, col) on the fp64 tensor path (four times the rate of the fp64 FMA pipe
// on this part).  Lane l holds a = A[l / 4][l % 4], b = B[l % 4][l / 4] and c0, c1 = D[l / 4][2 (l % 4) + {0, 1}].
__device__ __forceinline__ void dmma_8x8x4(double& c0, double& c1, double a, double b) {
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                 : "+d"(c0), "+d"(c1)
                 : "d"(a), "d"(b));
}

// T x T tile of S per CTA (T = 32; a multiple of 32), eight warps; a warp owns (T / 32) x (T / 16) fragments of 8 x 8 outputs.
// D goes through shared memory in chunks of 32 channels (row stride 36 doubles: the fragment loads then touch every
// bank pair twice, the minimum for 32 eight-byte lanes); the next chunk is fetched into registers while the
// current one is multiplied.  Every output accumulates its products in ascending order of the four-channel groups.
template <int T>
__global__ void __launch_bounds__(256) scores_kernel(const double* pooled, TensorGeom g, int n_img,
                                                     float* __restrict__ scores, const DevPlan* __restrict__ plan) {
    constexpr int NI = T / 32;           // 8-row fragments per warp
    constexpr int NJ = T / 16;           // 8-column fragments per warp
    constexpr int LD = T * 32 / 256;     // values a thread stages per operand and chunk
    constexpr int LDS = 36;              // row stride of the staged chunks in doubles
    __shared__ double sq[T][LDS];
    __shared__ double sk[T][LDS];
    const int ph = blockIdx.z;                       // p * H + h
    grid_dependency_launch();
    // The block means come from the kernel before, which may still be running when this one starts: wait for its end,
    // and read them past the L1 (ld.global.cg), whose lines no such wait is known to refresh.
    grid_dependency_wait();
    if (plan && ph >= plan->sparse.n * g.H) return;
    const int i0 = blockIdx.y * T, j0 = blockIdx.x * T;
    const double* pq = pooled + (long long)ph * g.nb * g.D;
    const double* pk = pooled + ((long long)n_img * g.H + ph) * g.nb * g.D;
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32, gr = lane >> 2, c = lane & 3;
    const int ri = (warp >> 1) * (8 * NI), cj = (warp & 1) * (8 * NJ);   // the warp's corner inside the tile
    double acc[NI][NJ][2];
#pragma unroll
    for (int a = 0; a < NI; ++a)
#pragma unroll
        for (int b = 0; b < NJ; ++b) acc[a][b][0] = acc[a][b][1] = 0.0;
    double rq[LD], rk[LD];
    auto fetch = [&](int d0) {
#pragma unroll
        for (int u = 0; u < LD; ++u) {
            const int e = threadIdx.x + u * 256, r = e / 32, cc = e % 32;
            rq[u] = (i0 + r < g.nb) ? __ldcg(pq + (long long)(i0 + r) * g.D + d0 + cc) : 0.0;
            rk[u] = (j0 + r < g.nb) ? __ldcg(pk + (long long)(j0 + r) * g.D + d0 + cc) : 0.0;
        }
    };
    fetch(0);
    for (int d0 = 0; d0 < g.D; d0 += 32) {
#pragma unroll
        for (int u = 0; u < LD; ++u) {
            const int e = threadIdx.x + u * 256, r = e / 32, cc = e % 32;
            sq[r][cc] = rq[u];
            sk[r][cc] = rk[u];
        }
        __syncthreads();
        if (d0 + 32 < g.D) fetch(d0 + 32);
#pragma unroll
        for (int d = 0; d < 32; d += 4) {
            double qa[NI], kb[NJ];
#pragma unroll
            for (int a = 0; a < NI; ++a) qa[a] = sq[ri + 8 * a + gr][d + c];
#pragma unroll
            for (int b = 0; b < NJ; ++b) kb[b] = sk[cj + 8 * b + gr][d + c];
#pragma unroll
            for (int a = 0; a < NI; ++a)
#pragma unroll
                for (int b = 0; b < NJ; ++b) dmma_8x8x4(acc[a][b][0], acc[a][b][1], qa[a], kb[b]);
        }
        __syncthreads();
    }
    float* so = scores + (long long)ph * g.nb * g.nb;
#pragma unroll
    for (int a = 0; a < NI; ++a)
#pragma unroll
        for (int b = 0; b < NJ; ++b)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int i = i0 + ri + 8 * a + gr, j = j0 + cj + 8 * b + 2 * c + e;
                if (i < g.nb && j < g.nb) so[(long long)i * g.nb + j] = (float)acc[a][b][e];
            }
}

}  // namespace

cudaError_t launch_block_pool(const void* q, const void* k, const TensorGeom& g, const ImgList& imgs,
                              double* pooled, cudaStream_t s, const DevPlan* plan, int n_cap) {
    if (!plan) n_cap = imgs.n;
    dim3 grid((g.nb + 3) / 4, g.H, 2 * n_cap);
    if (g.D == 128)
        pool_kernel<128><<<grid, 128, 0, s>>>((const uint16_t*)q, (const uint16_t*)k, g, imgs, pooled, plan, n_cap);
    else
        pool_kernel<64><<<grid, 128, 0, s>>>((const uint16_t*)q, (const uint16_t*)k, g, imgs, pooled, plan, n_cap);
    return cudaGetLastError();
}

cudaError_t launch_block_scores(const double* pooled, const TensorGeom& g, int n_img, float* scores,
                                cudaStream_t s, const DevPlan* plan, bool pdl) {
    // with a plan n_img is the capacity.  32 x 32 tiles at every length: against 64 x 64 tiles they waste less of
    // the ragged edge and fill the SMs more evenly (30 against 35 us at 264 blocks, where 64 x 64 pads 264 to 320)
    dim3 grid((g.nb + 31) / 32, (g.nb + 31) / 32, n_img * g.H);
    return launch_kernel(scores_kernel<32>, grid, dim3(256), 0, s, pdl, pooled, g, n_img, scores, plan);
}

// ---------------------------------------------------------------------------------------------
// rapid3_block_scores_static: the scoring pass for callers that may not allocate device memory.
//
// The block means (the only scratch of this pass) live in the file-scope array below instead of
// a cudaMalloc'ed workspace.  The array is part of the loaded module: every GPU that loads the
// library holds RAPID3_STATIC_SCRATCH_DOUBLES * 8 bytes (16 MiB) until the process exits.
// In host code the array's name is only a stand-in for the symbol, not a device address, so the
// address is looked up once per device with cudaGetSymbolAddress (with that device current) and
// that pointer is what the kernels get.
#include <mutex>

#define RAPID3_STATIC_SCRATCH_DOUBLES (1ll << 21)   // 16 MiB of fp64 block means
static __device__ __align__(256) double g_static_pool_scratch[RAPID3_STATIC_SCRATCH_DOUBLES];

namespace {

constexpr int RAPID3_STATIC_MAX_DEVICES = 64;

std::mutex g_static_mu;
double* g_static_ptr[RAPID3_STATIC_MAX_DEVICES] = {};

// Device address of the scratch array on the current device (looked up on first use per device).
int static_scratch(double** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= RAPID3_STATIC_MAX_DEVICES) return RAPID3_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_pool_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return RAPID3_ERR_CUDA;
        }
        g_static_ptr[dev] = static_cast<double*>(p);
    }
    *out = g_static_ptr[dev];
    return RAPID3_OK;
}

}  // namespace

extern "C" int rapid3_block_scores_static(const rapid3_shape* s, const void* q, const void* k,
                                          const int32_t* img_idx_host, int n_img, float* scores, void* stream) {
    if (!s || !q || !k || !scores) return RAPID3_ERR_INVALID_ARG;
    if (s->block != RAPID3_BLOCK || (s->D != 64 && s->D != 128)) return RAPID3_ERR_UNSUPPORTED;
    if (s->B_max < 1 || s->B_max > RAPID3_MAX_IMG || s->H < 1 || s->H > 65535) return RAPID3_ERR_INVALID_ARG;
    if ((long long)s->B_max * s->H > 65535) return RAPID3_ERR_UNSUPPORTED;     // (image, head) pairs index a grid dimension
    if (s->n_text < 0 || s->n_image < 0) return RAPID3_ERR_INVALID_ARG;
    const long long N = (long long)s->n_text + s->n_image;
    if (N < 1) return RAPID3_ERR_INVALID_ARG;
    if (N > 64ll * RAPID3_MAX_NB) return RAPID3_ERR_UNSUPPORTED;
    if (s->stride_n < s->D || s->stride_h < 1 || s->stride_b < 1) return RAPID3_ERR_INVALID_ARG;
    if ((s->stride_n % 8) || (s->stride_h % 8) || (s->stride_b % 8)) return RAPID3_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(q) % 16) || (reinterpret_cast<uintptr_t>(k) % 16)) return RAPID3_ERR_INVALID_ARG;
    if (n_img < 1 || n_img > s->B_max) return RAPID3_ERR_INVALID_ARG;

    TensorGeom g;
    g.H = s->H;
    g.D = s->D;
    g.N = (int)N;
    g.nb = (int)((N + 63) / 64);
    g.n_text_blocks = (s->n_text + 63) / 64;
    g.h0 = 0;
    g.pair_stride = 1;
    g.stride_b = s->stride_b;
    g.stride_h = s->stride_h;
    g.stride_n = s->stride_n;
    // block means of Q and K for the listed images must fit the fixed array
    const long long need = 2ll * n_img * g.H * g.nb * g.D;
    if (need > RAPID3_STATIC_SCRATCH_DOUBLES) return RAPID3_ERR_WORKSPACE;

    ImgList l;
    l.n = n_img;
    for (int p = 0; p < n_img; ++p) {
        const int b = img_idx_host ? img_idx_host[p] : p;
        if (b < 0 || b >= s->B_max) return RAPID3_ERR_INVALID_ARG;
        l.batch[p] = b;
        l.slot[p] = p;
        l.k_free[p] = 0;
    }
    double* scratch = nullptr;
    const int r = static_scratch(&scratch);
    if (r != RAPID3_OK) return r;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // every element of the used part of the scratch is written by the pooling kernel before the
    // scoring kernel reads it, so nothing has to be cleared between calls
    if (launch_block_pool(q, k, g, l, scratch, st) != cudaSuccess) return RAPID3_ERR_CUDA;
    if (launch_block_scores(scratch, g, n_img, scores, st, nullptr, true) != cudaSuccess) return RAPID3_ERR_CUDA;
    return RAPID3_OK;
}

extern "C" int64_t rapid3_static_scratch_bytes(void) { return RAPID3_STATIC_SCRATCH_DOUBLES * (int64_t)sizeof(double); }
