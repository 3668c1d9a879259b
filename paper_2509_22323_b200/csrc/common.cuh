// Shared declarations of the rapid3 CUDA library: launch-argument structs and the internal
// launcher prototypes.  Host API in api.cu; kernels in k1_scores.cu, k2_select.cu, k3_attn.cu.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "rapid3.h"

#define RAPID3_BLOCK 64
#define RAPID3_MAX_IMG 64     // images per launch (lists travel as kernel arguments)
#define RAPID3_MAX_NB 1024    // key blocks per sequence (65536 tokens)

// Per-launch image list.  batch[p]: index into the B dimension of Q/K/V/O.
// slot[p]: index into the compacted scores / mask / kept-list arrays, or -1 for a dense image.
// k_free[p]: free candidates kept per image row (select kernel).
struct ImgList {
    int n;
    int batch[RAPID3_MAX_IMG];
    int slot[RAPID3_MAX_IMG];
    int k_free[RAPID3_MAX_IMG];
};

// Device-resident plan of one gated step (filled by plan_kernel from device-resident actions):
// the two image lists the host path passes as kernel arguments.
struct DevPlan {
    ImgList sparse;   // images with keep ratio < 1, ascending batch order, slot = position
    ImgList all;      // every attending image, descending keep ratio (dense first)
    int n_dense;
};

// Keep counts per (sparse slot, head) for a policy that sets one ratio per head (Sec. 3.2: the
// sparsity head emits theta in R^{L x H}).  Travels as a kernel argument, so slots * H is bounded.
#define RAPID3_MAX_HEAD_ROWS 2048
struct HeadKeep {
    static constexpr int mode = 1;
    int k[RAPID3_MAX_HEAD_ROWS];
};
struct NoHeadKeep {
    static constexpr int mode = 0;
};
// Keep counts per row (image slot, head, query block) in device memory: the cumulative-mass rule
// arrives at a different count in every row.
struct RowKeep {
    static constexpr int mode = 2;
    const int32_t* k;
};
// Mass share tau per image of a launch (cumulative-mass selection).
struct MassShare {
    float tau[RAPID3_MAX_IMG];
};

struct TensorGeom {
    int H, D, N, nb, n_text_blocks;           // H: heads this launch covers
    int h0;                                   // first of them in the tensors (workspace arrays count heads from 0)
    int pair_stride;                          // 1, 2 or 3: which query blocks share an attention tile
    long long stride_b, stride_h, stride_n;   // elements
};

// Programmatic dependent launch: a kernel launched with `pdl` set may start while the kernel before it in the stream
// is still running, and must call grid_dependency_wait() before it touches anything that kernel writes; the kernel
// before it calls grid_dependency_launch() to let it start.  Both are no-ops in an ordinary launch.
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, bool pdl,
                                 Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// K1: block means of Q and K (fp64) for the listed images, then S = Qbar . Kbar^T -> fp32.
// With `plan` set the image list is read from device memory (plan->sparse) and the grid is sized
// for `n_cap` images; CTAs beyond the planned count return at once.  pooled is [2][n_cap][H][nb][D].
cudaError_t launch_block_pool(const void* q, const void* k, const TensorGeom& g, const ImgList& imgs,
                              double* pooled, cudaStream_t s, const DevPlan* plan = nullptr, int n_cap = 0);
// `pdl`: the kernel before it in the stream is this library's pooling kernel (same for the launchers below: the
// kernel named in their comment), so the launch may be a programmatic dependent one.
cudaError_t launch_block_scores(const double* pooled, const TensorGeom& g, int n_img, float* scores,
                                cudaStream_t s, const DevPlan* plan = nullptr, bool pdl = false);
// K2: forced + top-k selection.
cudaError_t launch_select_mask(const float* scores, const TensorGeom& g, const ImgList& imgs,
                               uint64_t* bitmask, int32_t* kept_idx, int32_t* kept_cnt, cudaStream_t s,
                               const DevPlan* plan = nullptr, int n_cap = 0, bool pdl = false);   // after the scores kernel
cudaError_t launch_select_mask_heads(const float* scores, const TensorGeom& g, const ImgList& imgs,
                                     const HeadKeep& hk, uint64_t* bitmask, int32_t* kept_idx, int32_t* kept_cnt,
                                     cudaStream_t s, bool pdl = false);                           // after the scores kernel
// K2, cumulative-mass variant: row_keep[row] = smallest count of best free candidates holding a share
// tau of the row's softmax mass (weights exp(scale * (S - row max)), fp64), then the top-k selection
// at that count.
cudaError_t launch_select_mask_mass(const float* scores, const TensorGeom& g, const ImgList& imgs,
                                    const MassShare& share, float scale, int32_t* row_keep, uint64_t* bitmask,
                                    int32_t* kept_idx, int32_t* kept_cnt, cudaStream_t s);
// K5: Q/K producer (RMS norm + gain + rotary embedding -> bf16) that also writes the block means of
// the images with a workspace slot.  pooled is [2][n_sparse][H][nb][D].
struct PrepArgs {
    const void* q_raw;
    const void* k_raw;
    void* q_out;
    void* k_out;
    const float* q_gain;
    const float* k_gain;
    const float* rot;     // [N][D/2][2] (cos, sin) or nullptr
    float eps;
};
cudaError_t launch_prepare(const PrepArgs& a, const TensorGeom& g, const ImgList& imgs, int n_sparse, double* pooled,
                           cudaStream_t s);
// Builds the plan from device-resident actions and keep ratios (one thread; B <= RAPID3_MAX_IMG).
cudaError_t launch_plan(const int32_t* action_dev, const float* ratio_dev, int B, const TensorGeom& g,
                        DevPlan* plan, int* status, cudaStream_t s);
// K3: attention over kept tiles.  `bitmask` (optional) is the select kernel's bitmask of the same
// lists; when present the kernel reads it instead of walking the lists.  inject_stop_group >= 0
// launches the failure-injection build of the kernel (see rapid3_debug_inject_timeout).
cudaError_t launch_attention(const CUtensorMap& tmq, const CUtensorMap& tmk, const CUtensorMap& tmv,
                             const CUtensorMap& tmo, const TensorGeom& g, const ImgList& imgs, const int32_t* kept_idx,
                             const int32_t* kept_cnt, const uint64_t* bitmask, float softmax_scale, int* status,
                             cudaStream_t s, const DevPlan* plan = nullptr, int n_cap = 0, int inject_stop_group = -1,
                             int pdl = 0);   // 1: after the selection kernel, whose masks only the sparse images' thread blocks read
cudaError_t attention_static_init();
