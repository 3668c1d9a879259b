// K4: the Cache-Reuse data path (paper Sec. 3.2 "Level-2: Cache-Reuse", the conditional
// definition of O_t): per image and step either the generator ran and its residual is cached,
//     delta = O - X            (action ATTEND: O is the generator's output, just computed)
// or the cached residual stands in for the generator,
//     O = X + delta            (action REUSE)
// and a skipped step touches nothing.  One launch covers the batch; the per-image action selects
// the branch.  bf16 in and out, the sum / difference taken in fp32 and rounded once to bf16.
// Pure streaming: 2 reads + 1 write of 16-byte vectors per 8 elements.
#include "common.cuh"

namespace {

struct CacheActions {
    int act[RAPID3_MAX_IMG];
};

__device__ __forceinline__ uint32_t addsub_bf16x2(uint32_t a, uint32_t b, float sign) {
    const float a0 = __uint_as_float(a << 16), a1 = __uint_as_float(a & 0xffff0000u);
    const float b0 = __uint_as_float(b << 16), b1 = __uint_as_float(b & 0xffff0000u);
    uint32_t d;
    const float r0 = fmaf(sign, b0, a0), r1 = fmaf(sign, b1, a1);     // a + sign * b, exact product
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(r1), "f"(r0));
    return d;
}

__global__ void __launch_bounds__(256) cache_step_kernel(const uint4* __restrict__ x, uint4* __restrict__ o,
                                                         uint4* __restrict__ delta, CacheActions acts,
                                                         long long vec_per_image) {
    const int b = blockIdx.y;
    const int a = acts.act[b];
    if (a == RAPID3_ACT_SKIP) return;
    const long long base = (long long)b * vec_per_image;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < vec_per_image;
         i += (long long)gridDim.x * blockDim.x) {
        const uint4 xv = __ldg(x + base + i);
        if (a == RAPID3_ACT_REUSE) {
            const uint4 dv = __ldg(delta + base + i);
            uint4 r;
            r.x = addsub_bf16x2(xv.x, dv.x, 1.f); r.y = addsub_bf16x2(xv.y, dv.y, 1.f);
            r.z = addsub_bf16x2(xv.z, dv.z, 1.f); r.w = addsub_bf16x2(xv.w, dv.w, 1.f);
            o[base + i] = r;
        } else {
            const uint4 ov = o[base + i];
            uint4 r;
            r.x = addsub_bf16x2(ov.x, xv.x, -1.f); r.y = addsub_bf16x2(ov.y, xv.y, -1.f);
            r.z = addsub_bf16x2(ov.z, xv.z, -1.f); r.w = addsub_bf16x2(ov.w, xv.w, -1.f);
            delta[base + i] = r;
        }
    }
}

}  // namespace

extern "C" int rapid3_cache_step(const void* x, void* o, void* delta, const int32_t* action_host, int B,
                                 int64_t elems_per_image, void* stream) {
    if (!x || !o || !delta || !action_host) return RAPID3_ERR_INVALID_ARG;
    if (B < 1 || B > RAPID3_MAX_IMG || elems_per_image < 8 || (elems_per_image % 8)) return RAPID3_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(x) % 16) || (reinterpret_cast<uintptr_t>(o) % 16) ||
        (reinterpret_cast<uintptr_t>(delta) % 16))
        return RAPID3_ERR_INVALID_ARG;
    CacheActions acts;
    bool any = false;
    for (int b = 0; b < B; ++b) {
        const int a = action_host[b];
        if (a != RAPID3_ACT_SKIP && a != RAPID3_ACT_REUSE && a != RAPID3_ACT_ATTEND) return RAPID3_ERR_INVALID_ARG;
        acts.act[b] = a;
        any = any || a != RAPID3_ACT_SKIP;
    }
    if (!any) return RAPID3_OK;                            // every image skipped: nothing is launched
    const long long vec = elems_per_image / 8;
    long long gx = (vec + 255) / 256;
    if (gx > 1184) gx = 1184;                              // 8 CTAs per SM on 148 SMs, grid-stride beyond
    dim3 grid((unsigned)gx, (unsigned)B);
    cache_step_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(x), static_cast<uint4*>(o), static_cast<uint4*>(delta), acts, vec);
    return cudaGetLastError() == cudaSuccess ? RAPID3_OK : RAPID3_ERR_CUDA;
}
