// K5: Q/K producer with the block pooling folded in.  Per-head RMS normalisation with a learned
// gain, rotary embedding (adjacent channel pairs, cos / sin per token from a caller-given table),
// one rounding to bf16 -- and, in the same pass, the fp64 block means of the ROUNDED values for the
// images that will be scored, so that the scoring pass does not have to read Q and K again.
// Layout of the work as in the pooling kernel: one warp per (Q|K, image, head, 64-token block), a
// token row of D channels is D / 8 lanes of 16 bytes; the row's sum of squares is reduced over
// those lanes with shuffles, the rotation is lane-local (a lane holds four whole pairs).
// HBM-bound: reads the raw Q and K once, writes Q and K once.
#include "common.cuh"

// Measured on FLUX 1024^2 shapes: two rows in flight per lane at six CTAs per SM (74 registers) beat deeper
// prefetch at lower occupancy; the kernel is bound by instruction issue and latency, not by the loads in flight.
#ifndef PREP_INFL
#define PREP_INFL 2
#endif
#ifndef PREP_MINB
#define PREP_MINB 6
#endif

namespace {

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

template <int D>
__global__ void __launch_bounds__(128, PREP_MINB) prepare_kernel(const uint16_t* __restrict__ q_raw,
                                                      const uint16_t* __restrict__ k_raw, uint16_t* q_out,
                                                      uint16_t* k_out, const float* __restrict__ q_gain,
                                                      const float* __restrict__ k_gain,
                                                      const float* __restrict__ rot, float eps, TensorGeom g,
                                                      ImgList imgs, int n_sparse, double* __restrict__ pooled) {
    constexpr int TPR = D / 8;          // lanes per token row (8 channels = 16 bytes each)
    constexpr int RPL = 32 / TPR;       // rows per warp-wide load
    constexpr int ITERS = 64 / RPL;     // loads per lane
    constexpr int INFL = PREP_INFL;     // rows in flight per lane
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int blk = blockIdx.x * 4 + warp, h = blockIdx.y;
    if (blk >= g.nb) return;
    const int which = blockIdx.z / imgs.n;            // 0 = Q, 1 = K
    const int p = blockIdx.z - which * imgs.n;
    const int batch = imgs.batch[p], slot = imgs.slot[p];
    const long long off = (long long)batch * g.stride_b + (long long)(g.h0 + h) * g.stride_h;
    const uint16_t* src = (which ? k_raw : q_raw) + off;
    uint16_t* dst = (which ? k_out : q_out) + off;
    const float* gain = which ? k_gain : q_gain;
    const int c = lane % TPR, r0 = lane / TPR;
    const int n0 = blk * 64;
    const int valid = min(64, g.N - n0);

    float gn[8];
    {
        const float4 g0 = __ldg(reinterpret_cast<const float4*>(gain + c * 8));
        const float4 g1 = __ldg(reinterpret_cast<const float4*>(gain + c * 8 + 4));
        gn[0] = g0.x; gn[1] = g0.y; gn[2] = g0.z; gn[3] = g0.w;
        gn[4] = g1.x; gn[5] = g1.y; gn[6] = g1.z; gn[7] = g1.w;
    }
    double acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.0;
#pragma unroll 1
    for (int it0 = 0; it0 < ITERS; it0 += INFL) {
        uint4 v[INFL];
        float4 cs[INFL][2];
#pragma unroll
        for (int u = 0; u < INFL; ++u) {
            const int row = (it0 + u) * RPL + r0;
            v[u] = make_uint4(0, 0, 0, 0);
            cs[u][0] = make_float4(1.f, 0.f, 1.f, 0.f);
            cs[u][1] = make_float4(1.f, 0.f, 1.f, 0.f);
            if (row < valid) {
                v[u] = __ldg(reinterpret_cast<const uint4*>(src + (long long)(n0 + row) * g.stride_n + c * 8));
                if (rot) {
                    const float4* rp = reinterpret_cast<const float4*>(rot + ((long long)(n0 + row) * (D / 2) + c * 4) * 2);
                    cs[u][0] = __ldg(rp);
                    cs[u][1] = __ldg(rp + 1);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < INFL; ++u) {
            const int row = (it0 + u) * RPL + r0;
            float x[8] = {bf16_lo(v[u].x), bf16_hi(v[u].x), bf16_lo(v[u].y), bf16_hi(v[u].y),
                          bf16_lo(v[u].z), bf16_hi(v[u].z), bf16_lo(v[u].w), bf16_hi(v[u].w)};
            float ss = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) ss = fmaf(x[e], x[e], ss);
#pragma unroll
            for (int o = 1; o < TPR; o <<= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
            const float r = rsqrtf(ss * (1.0f / (float)D) + eps);       // 2 ulp: far inside the bf16 rounding of the result
#pragma unroll
            for (int e = 0; e < 8; ++e) x[e] = x[e] * r * gn[e];
            const float cz[4] = {cs[u][0].x, cs[u][0].z, cs[u][1].x, cs[u][1].z};
            const float sz[4] = {cs[u][0].y, cs[u][0].w, cs[u][1].y, cs[u][1].w};
            uint32_t w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float z0 = x[2 * i] * cz[i] - x[2 * i + 1] * sz[i];
                const float z1 = x[2 * i] * sz[i] + x[2 * i + 1] * cz[i];
                w[i] = pack2(z0, z1);
            }
            if (row < valid) {
                *reinterpret_cast<uint4*>(dst + (long long)(n0 + row) * g.stride_n + c * 8) =
                    make_uint4(w[0], w[1], w[2], w[3]);
                if (slot >= 0) {                              // only scored images need their block means
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        acc[2 * i] += (double)bf16_lo(w[i]);
                        acc[2 * i + 1] += (double)bf16_hi(w[i]);
                    }
                }
            }
        }
    }
    if (slot < 0) return;                             // a dense image is not scored (warp-uniform)
#pragma unroll
    for (int o = TPR; o < 32; o <<= 1)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
    if (lane < TPR) {
        double* o = pooled + ((((long long)which * n_sparse + slot) * g.H + h) * g.nb + blk) * D + c * 8;
        const double inv = 1.0 / (double)valid;
#pragma unroll
        for (int e = 0; e < 8; e += 2) *reinterpret_cast<double2*>(o + e) = make_double2(acc[e] * inv, acc[e + 1] * inv);
    }
}

}  // namespace

cudaError_t launch_prepare(const PrepArgs& a, const TensorGeom& g, const ImgList& imgs, int n_sparse, double* pooled,
                           cudaStream_t s) {
    dim3 grid((g.nb + 3) / 4, g.H, 2 * imgs.n);
    const uint16_t* qr = static_cast<const uint16_t*>(a.q_raw);
    const uint16_t* kr = static_cast<const uint16_t*>(a.k_raw);
    uint16_t* qo = static_cast<uint16_t*>(a.q_out);
    uint16_t* ko = static_cast<uint16_t*>(a.k_out);
    if (g.D == 128)
        prepare_kernel<128><<<grid, 128, 0, s>>>(qr, kr, qo, ko, a.q_gain, a.k_gain, a.rot, a.eps, g, imgs, n_sparse, pooled);
    else
        prepare_kernel<64><<<grid, 128, 0, s>>>(qr, kr, qo, ko, a.q_gain, a.k_gain, a.rot, a.eps, g, imgs, n_sparse, pooled);
    return cudaGetLastError();
}
