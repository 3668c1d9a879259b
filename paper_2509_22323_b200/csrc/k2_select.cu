// K2: per (image, head, query-block row) forced + top-k block selection.
// One warp per row.  The row of fp32 scores is staged in shared memory; every free candidate
// gets its rank by counting the candidates that beat it under (score descending, index
// ascending); rank < k keeps it.  The bitmask is assembled with warp ballots and the ascending
// kept list with ballot prefix counts, so the row is written in one pass.
#include "common.cuh"

namespace {

constexpr int WARPS = 4;

__global__ void __launch_bounds__(WARPS * 32) select_kernel(const float* __restrict__ scores, TensorGeom g,
                                                            ImgList imgs, uint32_t* __restrict__ bitmask32,
                                                            int32_t* __restrict__ kept_idx,
                                                            int32_t* __restrict__ kept_cnt, int words32) {
    extern __shared__ float srow[];                       // [WARPS][nb_pad]
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int nb = g.nb, ntb = g.n_text_blocks;
    const int nb_pad = (nb + 31) & ~31;
    const long long row = (long long)blockIdx.x * WARPS + warp;        // (p * H + h) * nb + i
    const long long n_rows = (long long)imgs.n * g.H * nb;
    if (row >= n_rows) return;
    const int i = (int)(row % nb);
    const int p = (int)(row / ((long long)nb * g.H));
    const int k = imgs.k_free[p];
    float* s = srow + warp * nb_pad;
    const float* src = scores + row * nb;
    for (int j = lane; j < nb; j += 32) s[j] = src[j];
    __syncwarp();

    const bool text_row = i < ntb;
    int32_t* out_idx = kept_idx + row * nb;
    uint32_t* out_bits = bitmask32 + row * words32;
    int total = 0;
    for (int c = 0; c < nb_pad; c += 32) {
        const int j = c + lane;
        bool keep = false;
        if (j < nb) {
            if (text_row || j < ntb || j == i) {
                keep = true;
            } else {
                const float sj = s[j];
                int rank = 0;
                for (int m = ntb; m < nb; ++m) {
                    const float sm = s[m];
                    rank += (m != i) && (sm > sj || (sm == sj && m < j));
                }
                keep = rank < k;
            }
        }
        const uint32_t bal = __ballot_sync(0xffffffffu, keep);
        if (lane == 0) out_bits[c / 32] = bal;
        if (keep) out_idx[total + __popc(bal & ((1u << lane) - 1u))] = j;
        total += __popc(bal);
    }
    for (int c = nb_pad / 32 + lane; c < words32; c += 32) out_bits[c] = 0;   // odd 32-bit half of the last word
    for (int e = total + lane; e < nb; e += 32) out_idx[e] = -1;
    if (lane == 0) kept_cnt[row] = total;
}

}  // namespace

cudaError_t launch_select_mask(const float* scores, const TensorGeom& g, const ImgList& imgs, uint64_t* bitmask,
                               int32_t* kept_idx, int32_t* kept_cnt, cudaStream_t s) {
    const long long n_rows = (long long)imgs.n * g.H * g.nb;
    const int nb_pad = (g.nb + 31) & ~31;
    const int words32 = 2 * ((g.nb + 63) / 64);
    const unsigned grid = (unsigned)((n_rows + WARPS - 1) / WARPS);
    const size_t smem = (size_t)WARPS * nb_pad * sizeof(float);
    select_kernel<<<grid, WARPS * 32, smem, s>>>(scores, g, imgs, reinterpret_cast<uint32_t*>(bitmask), kept_idx,
                                                 kept_cnt, words32);
    return cudaGetLastError();
}
