// K2: per (image, head, query-block row) forced + top-k block selection.
// One warp per row.  The row of fp32 scores is staged in shared memory as order-preserving
// 32-bit keys.  The k-th largest free candidate is found by a radix select over the key bits
// (the bits all candidates share are skipped, the others go eight at a time through a 256-bin
// histogram and a scan from the top; rows with at most 32 candidates rank each candidate by
// counting the 64-bit (key, index) composites that beat it instead); a free
// candidate is kept when its key is above that threshold, or equal to it and among the first
// (lowest block index) of the equal ones still needed -- the order "score descending, index
// ascending".  The bitmask is assembled with warp ballots and the ascending kept list with ballot
// prefix counts, so the row is written in one pass.
#include "common.cuh"

namespace {

constexpr int WARPS = 4;

// HK = NoHeadKeep: one keep count per image.  HK = HeadKeep: one per (image, head), passed by value.
// HK = RowKeep: one per row, read from device memory.
template <typename HK>
__global__ void __launch_bounds__(WARPS * 32) select_kernel(const float* scores, TensorGeom g,
                                                            ImgList imgs, uint32_t* __restrict__ bitmask32,
                                                            int32_t* __restrict__ kept_idx,
                                                            int32_t* __restrict__ kept_cnt, int words32,
                                                            const DevPlan* __restrict__ plan, const HK hk) {
    extern __shared__ unsigned long long srow[];          // [WARPS][nb_pad] 64-bit slots, then [WARPS][256] histogram bins
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int nb = g.nb, ntb = g.n_text_blocks;
    const int nb_pad = (nb + 31) & ~31;
    const long long row = (long long)blockIdx.x * WARPS + warp;        // (p * H + h) * nb + i
    grid_dependency_launch();
    grid_dependency_wait();                             // the scores come from the kernel before, which may still be running
    const long long n_rows = (long long)(plan ? plan->sparse.n : imgs.n) * g.H * nb;
    if (row >= n_rows) return;
    const int i = (int)(row % nb);
    const int p = (int)(row / ((long long)nb * g.H));
    // free candidates kept in this row: one count per image, or per (image, head) when the policy
    // sets a ratio for every head
    int k;
    if constexpr (HK::mode == 1) k = hk.k[p * g.H + (int)((row / nb) % g.H)];
    else if constexpr (HK::mode == 2) k = hk.k[row];
    else k = plan ? plan->sparse.k_free[p] : imgs.k_free[p];
    // long rows keep 32-bit keys in the slots' memory, short rows 64-bit (key, index) composites
    unsigned long long* c64 = srow + warp * nb_pad;
    uint32_t* s = reinterpret_cast<uint32_t*>(c64);
    const float* src = scores + row * nb;
    const bool text_row = i < ntb;
    const int n_free = max(nb - ntb - ((i >= ntb) ? 1 : 0), 0);
    const bool select = !text_row && k > 0 && k < n_free;
    const bool radix = n_free > 32;                     // short rows: ranking by counting is cheaper (measured: 63 candidates already favour the histogram)
    // key: unsigned integer with the same order as the float (-0 and +0 made equal), at least 2^23 for
    // any finite score.  Forced blocks and padding get key 0: they match no radix prefix (every trial
    // prefix has a bit set) and beat no candidate, so the loops below need no index tests.
    for (int j = lane; j < nb_pad; j += 32) {
        uint32_t u = 0u;
        if (j < nb && j >= ntb && j != i) {
            u = __float_as_uint(__ldcg(src + j));              // past the L1: see the wait above
            if (u == 0x80000000u) u = 0u;
            u ^= (u >> 31) ? 0xffffffffu : 0x80000000u;
        }
        // composite: equal scores rank by ascending block index, so no two candidates compare equal
        if (radix) s[j] = u;
        else c64[j] = u ? (((unsigned long long)u << 32) | (uint32_t)(0xffffffffu - (uint32_t)j)) : 0ull;
    }
    __syncwarp();
    // radix select of the k-th largest key among the free candidates: the bits all candidates share are skipped,
    // the rest is taken eight bits at a time, each round a 256-bin histogram of the candidates that still match
    // the prefix (shared-memory atomics) and a scan over the bins from the top
    uint32_t prefix = 0u;
    int want = k;                                       // rank still looked for inside the prefix group
    if (select && radix) {
        uint32_t* hist = reinterpret_cast<uint32_t*>(srow + WARPS * nb_pad) + warp * 256;
        uint32_t k_and = 0xffffffffu, k_or = 0u;
        for (int j = lane; j < nb_pad; j += 32) {
            const uint32_t u = s[j];
            if (u) { k_and &= u; k_or |= u; }
        }
        k_and = __reduce_and_sync(0xffffffffu, k_and);
        k_or = __reduce_or_sync(0xffffffffu, k_or);
        const uint32_t diff = k_and ^ k_or;             // bits in which two candidates differ
        const int top = diff ? 32 - __clz(diff) : 0;    // only bits below `top` can differ
        prefix = top >= 32 ? 0u : (k_or & ~((1u << top) - 1u));
        for (int hi = top; hi > 0; hi -= 8) {           // digit = bits [lo, hi)
            const int lo = max(hi - 8, 0);
            const uint32_t dmask = (1u << (hi - lo)) - 1u;
#pragma unroll
            for (int b = 0; b < 8; ++b) hist[8 * lane + b] = 0u;
            __syncwarp();
            for (int j = lane; j < nb_pad; j += 32) {
                const uint32_t u = s[j];
                if (u && (hi >= 32 || (u >> hi) == (prefix >> hi))) atomicAdd(&hist[(u >> lo) & dmask], 1u);
            }
            __syncwarp();
            // lane l owns bins 8 l .. 8 l + 7; S = candidates in its bins and all higher ones
            uint32_t hloc[8], T = 0u;
#pragma unroll
            for (int b = 0; b < 8; ++b) {
                hloc[b] = hist[8 * lane + b];
                T += hloc[b];
            }
            uint32_t S = T;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t v = __shfl_down_sync(0xffffffffu, S, o);
                if (lane + o < 32) S += v;
            }
            const int L = 31 - __clz(__ballot_sync(0xffffffffu, S >= (uint32_t)want));   // the lane whose bins hold the rank
            int d_loc = -1;
            uint32_t above_loc = 0u, running = S - T;
#pragma unroll
            for (int b = 7; b >= 0; --b) {
                if (d_loc < 0 && running + hloc[b] >= (uint32_t)want) {
                    d_loc = b;
                    above_loc = running;
                }
                running += hloc[b];
            }
            const int d = __shfl_sync(0xffffffffu, 8 * lane + d_loc, L);
            const uint32_t above = __shfl_sync(0xffffffffu, above_loc, L);
            prefix |= (uint32_t)d << lo;
            want -= (int)above;
            __syncwarp();
        }
    }
    int32_t* out_idx = kept_idx + row * nb;
    uint32_t* out_bits = bitmask32 + row * words32;
    int total = 0, eq_seen = 0;
    for (int c = 0; c < nb_pad; c += 32) {
        const int j = c + lane;
        bool keep = false, eq = false;
        if (j < nb) {
            if (text_row || j < ntb || j == i) {
                keep = true;
            } else if (select && radix) {
                keep = s[j] > prefix;
                eq = s[j] == prefix;
            } else if (select) {
                // rank = number of free candidates that beat this one (key descending, index ascending)
                const unsigned long long cj = c64[j];
                int rank = 0;
#pragma unroll 4
                for (int m = ntb; m < nb; ++m) rank += c64[m] > cj;
                keep = rank < k;
            } else {
                keep = k >= n_free && k > 0;            // every free candidate, or none
            }
        }
        // equal keys: the lowest block indices first, `want` of them in all
        const uint32_t beq = __ballot_sync(0xffffffffu, eq);
        if (eq && eq_seen + __popc(beq & ((1u << lane) - 1u)) < want) keep = true;
        eq_seen += __popc(beq);
        const uint32_t bal = __ballot_sync(0xffffffffu, keep);
        if (lane == 0) out_bits[c / 32] = bal;
        if (keep) out_idx[total + __popc(bal & ((1u << lane) - 1u))] = j;
        total += __popc(bal);
    }
    for (int c = nb_pad / 32 + lane; c < words32; c += 32) out_bits[c] = 0;   // odd 32-bit half of the last word
    for (int e = total + lane; e < nb; e += 32) out_idx[e] = -1;
    if (lane == 0) kept_cnt[row] = total;
}

// Cumulative-mass rule: one warp per row finds the smallest count k of best free candidates (score
// descending, index ascending) whose weights w = exp(scale * (S - row max)) sum to at least
// tau * (sum of all free weights).  No sort: the boundary candidate is found by descending the
// bits of the order-preserving keys, each round summing the weights of the candidates that match
// the trial prefix (a weighted radix select); candidates equal to the boundary key are then added
// one by one.  fp64 throughout, the precision in which the decision is defined.
constexpr int MASS_WARPS = 2;

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__global__ void __launch_bounds__(MASS_WARPS * 32) mass_count_kernel(const float* __restrict__ scores, TensorGeom g,
                                                                     int n_img, MassShare share, float scale,
                                                                     int32_t* __restrict__ row_keep) {
    extern __shared__ double mass_smem[];                  // [MASS_WARPS][nb_pad] weights, then the keys
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int nb = g.nb, ntb = g.n_text_blocks;
    const int nb_pad = (nb + 31) & ~31;
    const long long row = (long long)blockIdx.x * MASS_WARPS + warp;
    if (row >= (long long)n_img * g.H * nb) return;
    const int i = (int)(row % nb);
    const int p = (int)(row / ((long long)nb * g.H));
    const int n_free = (i < ntb) ? 0 : max(nb - ntb - 1, 0);
    const float tau = share.tau[p];
    if (n_free == 0 || tau >= 1.f) {                       // warp-uniform
        if (lane == 0) row_keep[row] = n_free;
        return;
    }
    double* w = mass_smem + warp * nb_pad;
    uint32_t* key = reinterpret_cast<uint32_t*>(mass_smem + MASS_WARPS * nb_pad) + warp * nb_pad;
    const float* src = scores + row * nb;
    float mx = -INFINITY;
    for (int j = lane; j < nb; j += 32)
        if (j >= ntb && j != i) mx = fmaxf(mx, src[j]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    double part = 0.0;
    for (int j = lane; j < nb_pad; j += 32) {
        const bool is_free = j < nb && j >= ntb && j != i;
        uint32_t u = 0u;
        double wj = 0.0;
        if (is_free) {
            const float sj = src[j];
            u = __float_as_uint(sj);
            if (u == 0x80000000u) u = 0u;
            u ^= (u >> 31) ? 0xffffffffu : 0x80000000u;
            wj = exp((double)scale * ((double)sj - (double)mx));
        }
        key[j] = u;
        w[j] = wj;                                         // forced and padding entries weigh nothing
        part += wj;
    }
    __syncwarp();
    const double total = warp_sum(part);
    double want = (double)tau * total;                     // mass still to be covered inside the prefix group
    uint32_t prefix = 0u, mask = 0u;
    for (int bit = 31; bit >= 0; --bit) {
        const uint32_t trial = prefix | (1u << bit), m2 = mask | (1u << bit);
        double m1 = 0.0;
        for (int j = lane; j < nb_pad; j += 32) m1 += ((key[j] & m2) == trial) ? w[j] : 0.0;
        m1 = warp_sum(m1);
        if (m1 >= want) prefix = trial;
        else want -= m1;
        mask = m2;
    }
    // candidates above the boundary key are all kept; those equal to it one by one until the mass is reached
    int n_gt = 0, n_eq = 0;
    double w_eq = 0.0;
    for (int j = lane; j < nb; j += 32) {
        const bool is_free = j >= ntb && j != i;
        n_gt += is_free && key[j] > prefix;
        if (is_free && key[j] == prefix) {
            ++n_eq;
            w_eq = w[j];
        }
    }
    n_gt = __reduce_add_sync(0xffffffffu, n_gt);
    n_eq = __reduce_add_sync(0xffffffffu, n_eq);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) w_eq = fmax(w_eq, __shfl_xor_sync(0xffffffffu, w_eq, o));
    int r = 0;
    double acc = 0.0;
    while (r < n_eq && (r == 0 || acc < want)) {
        acc += w_eq;
        ++r;
    }
    if (lane == 0) row_keep[row] = min(max(n_gt + r, 1), n_free);
}

}  // namespace

cudaError_t launch_select_mask_mass(const float* scores, const TensorGeom& g, const ImgList& imgs,
                                    const MassShare& share, float scale, int32_t* row_keep, uint64_t* bitmask,
                                    int32_t* kept_idx, int32_t* kept_cnt, cudaStream_t s) {
    const long long n_rows = (long long)imgs.n * g.H * g.nb;
    const int nb_pad = (g.nb + 31) & ~31;
    {
        const unsigned grid = (unsigned)((n_rows + MASS_WARPS - 1) / MASS_WARPS);
        const size_t smem = (size_t)MASS_WARPS * nb_pad * (sizeof(double) + sizeof(uint32_t));
        mass_count_kernel<<<grid, MASS_WARPS * 32, smem, s>>>(scores, g, imgs.n, share, scale, row_keep);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    const int words32 = 2 * ((g.nb + 63) / 64);
    const unsigned grid = (unsigned)((n_rows + WARPS - 1) / WARPS);
    const size_t smem = (size_t)WARPS * nb_pad * sizeof(unsigned long long) + WARPS * 256 * sizeof(uint32_t);
    RowKeep rk;
    rk.k = row_keep;
    select_kernel<RowKeep><<<grid, WARPS * 32, smem, s>>>(scores, g, imgs, reinterpret_cast<uint32_t*>(bitmask), kept_idx,
                                                          kept_cnt, words32, nullptr, rk);
    return cudaGetLastError();
}

cudaError_t launch_select_mask(const float* scores, const TensorGeom& g, const ImgList& imgs, uint64_t* bitmask,
                               int32_t* kept_idx, int32_t* kept_cnt, cudaStream_t s, const DevPlan* plan, int n_cap,
                               bool pdl) {
    const long long n_rows = (long long)(plan ? n_cap : imgs.n) * g.H * g.nb;
    const int nb_pad = (g.nb + 31) & ~31;
    const int words32 = 2 * ((g.nb + 63) / 64);
    const unsigned grid = (unsigned)((n_rows + WARPS - 1) / WARPS);
    const size_t smem = (size_t)WARPS * nb_pad * sizeof(unsigned long long) + WARPS * 256 * sizeof(uint32_t);
    return launch_kernel(select_kernel<NoHeadKeep>, dim3(grid), dim3(WARPS * 32), smem, s, pdl, scores, g, imgs,
                         reinterpret_cast<uint32_t*>(bitmask), kept_idx, kept_cnt, words32, plan, NoHeadKeep());
}

cudaError_t launch_select_mask_heads(const float* scores, const TensorGeom& g, const ImgList& imgs, const HeadKeep& hk,
                                     uint64_t* bitmask, int32_t* kept_idx, int32_t* kept_cnt, cudaStream_t s, bool pdl) {
    const long long n_rows = (long long)imgs.n * g.H * g.nb;
    const int nb_pad = (g.nb + 31) & ~31;
    const int words32 = 2 * ((g.nb + 63) / 64);
    const unsigned grid = (unsigned)((n_rows + WARPS - 1) / WARPS);
    const size_t smem = (size_t)WARPS * nb_pad * sizeof(unsigned long long) + WARPS * 256 * sizeof(uint32_t);
    return launch_kernel(select_kernel<HeadKeep>, dim3(grid), dim3(WARPS * 32), smem, s, pdl, scores, g, imgs,
                         reinterpret_cast<uint32_t*>(bitmask), kept_idx, kept_cnt, words32, static_cast<const DevPlan*>(nullptr), hk);
}


// ---------------------------------------------------------------------------------------------
// Plan of a gated step from device-resident policy actions: the gate and compaction the host
// entry point does on the CPU, for callers whose sampled actions never leave the GPU.
namespace {

__global__ void plan_kernel(const int32_t* __restrict__ action, const float* __restrict__ ratio, int B, int n_free_img,
                            DevPlan* __restrict__ plan, int* __restrict__ status) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    ImgList& sp = plan->sparse;
    ImgList& al = plan->all;
    sp.n = 0;
    al.n = 0;
    int n_dense = 0;
    float ratio_of[RAPID3_MAX_IMG];
    for (int b = 0; b < B; ++b) {
        const int a = action[b];
        if (a != RAPID3_ACT_SKIP && a != RAPID3_ACT_REUSE && a != RAPID3_ACT_ATTEND) {
            atomicExch(status, RAPID3_ERR_INVALID_ARG);       // unknown action: treated as a skip
            continue;
        }
        if (a != RAPID3_ACT_ATTEND) continue;
        const float r = ratio[b];
        if (!(r > 0.f) || !(r <= 1.f)) {
            atomicExch(status, RAPID3_ERR_INVALID_ARG);       // ratio outside (0, 1]: image not processed
            continue;
        }
        int slot = -1;
        if (r < 1.f) {
            slot = sp.n++;
            sp.batch[slot] = b;
            sp.slot[slot] = slot;
            double x = ceil((double)r * (double)n_free_img - 1e-6);
            x = x < 0.0 ? 0.0 : (x > (double)n_free_img ? (double)n_free_img : x);
            sp.k_free[slot] = (int)x;
        } else {
            ++n_dense;
        }
        int pos = al.n++;
        while (pos > 0 && ratio_of[pos - 1] < r) {            // insertion sort, descending ratio, stable
            al.batch[pos] = al.batch[pos - 1];
            al.slot[pos] = al.slot[pos - 1];
            ratio_of[pos] = ratio_of[pos - 1];
            --pos;
        }
        al.batch[pos] = b;
        al.slot[pos] = slot;
        al.k_free[pos] = 0;
        ratio_of[pos] = r;
    }
    plan->n_dense = n_dense;
}

}  // namespace

cudaError_t launch_plan(const int32_t* action_dev, const float* ratio_dev, int B, const TensorGeom& g, DevPlan* plan,
                        int* status, cudaStream_t s) {
    const int n_free_img = g.nb - g.n_text_blocks - 1;
    plan_kernel<<<1, 32, 0, s>>>(action_dev, ratio_dev, B, n_free_img > 0 ? n_free_img : 0, plan, status);
    return cudaGetLastError();
}
