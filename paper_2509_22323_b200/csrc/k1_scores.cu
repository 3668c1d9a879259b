// K1: pooled block scores.
//   pool_kernel   : one CTA per (Q|K, image, head, 64-token block); 128-bit coalesced loads,
//                   fp64 accumulation (the sum of <= 64 bf16 values is exact in fp64), mean over
//                   the valid tokens of the block.  HBM-bound: reads Q and K exactly once.
//   scores_kernel : S[i][j] = Qbar[i,:] . Kbar[j,:] in fp64, rounded once to fp32.
#include "common.cuh"

namespace {

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

template <int D>
__global__ void __launch_bounds__(256) pool_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k,
                                                   TensorGeom g, ImgList imgs, double* __restrict__ pooled) {
    constexpr int TPR = D / 8;          // threads per token row (8 channels = 16 bytes each)
    constexpr int RG = 256 / TPR;       // row groups
    constexpr int RPT = 64 / RG;        // rows per thread
    __shared__ double red[RG][D + 1];

    const int blk = blockIdx.x, h = blockIdx.y;
    const int which = blockIdx.z / imgs.n;            // 0 = Q, 1 = K
    const int p = blockIdx.z - which * imgs.n;
    const uint16_t* base = (which ? k : q) + (long long)imgs.batch[p] * g.stride_b + (long long)h * g.stride_h;
    const int t = threadIdx.x, c = t % TPR, rg = t / TPR;
    const int n0 = blk * 64;
    const int valid = min(64, g.N - n0);

    uint4 v[RPT];
#pragma unroll
    for (int r = 0; r < RPT; ++r) {
        int row = rg + r * RG;
        v[r] = make_uint4(0, 0, 0, 0);
        if (row < valid)
            v[r] = __ldg(reinterpret_cast<const uint4*>(base + (long long)(n0 + row) * g.stride_n + c * 8));
    }
    double acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.0;
#pragma unroll
    for (int r = 0; r < RPT; ++r) {
        acc[0] += (double)bf16_lo(v[r].x); acc[1] += (double)bf16_hi(v[r].x);
        acc[2] += (double)bf16_lo(v[r].y); acc[3] += (double)bf16_hi(v[r].y);
        acc[4] += (double)bf16_lo(v[r].z); acc[5] += (double)bf16_hi(v[r].z);
        acc[6] += (double)bf16_lo(v[r].w); acc[7] += (double)bf16_hi(v[r].w);
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) red[rg][c * 8 + e] = acc[e];
    __syncthreads();
    if (t < D) {
        double s = 0.0;
#pragma unroll 8
        for (int r = 0; r < RG; ++r) s += red[r][t];
        long long o = ((((long long)which * imgs.n + p) * g.H + h) * g.nb + blk) * D + t;
        pooled[o] = s / (double)valid;
    }
}

// 32 x 32 tile of S per CTA, 16 x 16 threads, 2 x 2 outputs per thread, D in chunks of 32.
__global__ void __launch_bounds__(256) scores_kernel(const double* __restrict__ pooled, TensorGeom g, int n_img,
                                                     float* __restrict__ scores) {
    __shared__ double sq[32][33];
    __shared__ double sk[32][33];
    const int ph = blockIdx.z;                       // p * H + h
    const int i0 = blockIdx.y * 32, j0 = blockIdx.x * 32;
    const double* pq = pooled + (long long)ph * g.nb * g.D;
    const double* pk = pooled + ((long long)n_img * g.H + ph) * g.nb * g.D;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    double a00 = 0, a01 = 0, a10 = 0, a11 = 0;
    for (int d0 = 0; d0 < g.D; d0 += 32) {
        for (int e = threadIdx.x; e < 32 * 32; e += 256) {
            int r = e / 32, c = e % 32;
            sq[r][c] = (i0 + r < g.nb) ? pq[(long long)(i0 + r) * g.D + d0 + c] : 0.0;
            sk[r][c] = (j0 + r < g.nb) ? pk[(long long)(j0 + r) * g.D + d0 + c] : 0.0;
        }
        __syncthreads();
#pragma unroll 8
        for (int d = 0; d < 32; ++d) {
            double q0 = sq[ty][d], q1 = sq[ty + 16][d], k0 = sk[tx][d], k1 = sk[tx + 16][d];
            a00 += q0 * k0; a01 += q0 * k1; a10 += q1 * k0; a11 += q1 * k1;
        }
        __syncthreads();
    }
    float* so = scores + (long long)ph * g.nb * g.nb;
    int i = i0 + ty, j = j0 + tx;
    if (i < g.nb && j < g.nb) so[(long long)i * g.nb + j] = (float)a00;
    if (i < g.nb && j + 16 < g.nb) so[(long long)i * g.nb + j + 16] = (float)a01;
    if (i + 16 < g.nb && j < g.nb) so[(long long)(i + 16) * g.nb + j] = (float)a10;
    if (i + 16 < g.nb && j + 16 < g.nb) so[(long long)(i + 16) * g.nb + j + 16] = (float)a11;
}

}  // namespace

cudaError_t launch_block_pool(const void* q, const void* k, const TensorGeom& g, const ImgList& imgs,
                              double* pooled, cudaStream_t s) {
    dim3 grid(g.nb, g.H, 2 * imgs.n);
    if (g.D == 128)
        pool_kernel<128><<<grid, 256, 0, s>>>((const uint16_t*)q, (const uint16_t*)k, g, imgs, pooled);
    else
        pool_kernel<64><<<grid, 256, 0, s>>>((const uint16_t*)q, (const uint16_t*)k, g, imgs, pooled);
    return cudaGetLastError();
}

cudaError_t launch_block_scores(const double* pooled, const TensorGeom& g, int n_img, float* scores,
                                cudaStream_t s) {
    dim3 grid((g.nb + 31) / 32, (g.nb + 31) / 32, n_img * g.H);
    scores_kernel<<<grid, 256, 0, s>>>(pooled, g, n_img, scores);
    return cudaGetLastError();
}
