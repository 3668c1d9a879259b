// K3: masked flash-style joint attention over the kept key tiles (sm_100a).
//
// One CTA per (image, head, pair of adjacent 64-token query blocks) = a 128-row Q tile, the
// native UMMA M.  The two query blocks' ascending kept lists are merged into one union list;
// the CTA walks it two key blocks (128 keys) at a time.  A 64x64 sub-tile whose key block is
// not in that query block's own list is masked out before the softmax, so each query block
// attends exactly its own kept set.
//
// Roles (192 threads):
//   warps 0-3  softmax: thread = one query row; S from TMEM (tcgen05.ld), fp32 online softmax
//              with lazy rescale, P written back to TMEM as bf16 (aliasing S), final O / l store
//   warp 4     producer: TMA loads (cp.async.bulk.tensor, 128-byte swizzle) of Q once and of
//              gathered K / V key blocks per tile
//   warp 5     TMEM allocation and UMMA issue: S = Q K^T (both operands in shared memory),
//              O += P V (P from TMEM, V from shared memory as an N-major operand)
// Two CTAs are resident per SM (2 x 256 TMEM columns, ~100 KB shared memory each) so one CTA's
// softmax overlaps the other's MMAs.  Every mbarrier wait is bounded; a wait that runs out
// records RAPID3_ERR_TIMEOUT in the status word and the CTA drains and exits normally.
#include "common.cuh"
#include "ptx.cuh"

using namespace ptx;

namespace {

constexpr int NTHREADS = 192;
constexpr int TMEM_COLS = 256;
constexpr int S_COL = 0;
constexpr int O_COL = 128;
constexpr int HALF_BYTES = 16384;   // one 64-channel half of a 128-row tile: 128 rows x 128 bytes
constexpr int BLK_BYTES = 8192;     // 64 rows x 128 bytes
constexpr float RESCALE_LOG2 = 8.0f;

struct AttnParams {
    TensorGeom g;
    ImgList imgs;
    const int32_t* kept_idx;
    const int32_t* kept_cnt;
    uint16_t* out;
    int* status;
    float scale_log2;
};

enum { BAR_Q_FULL = 0, BAR_K_FULL, BAR_K_EMPTY, BAR_V_FULL, BAR_V_EMPTY, BAR_S_FULL, BAR_P_FULL, BAR_PV_DONE, N_BARS };

struct __align__(16) Ctl {
    unsigned long long bars[N_BARS];
    uint32_t tmem_base;
    int n_u;
    volatile int abort_flag;
    uint32_t bm[2][32];
    int16_t u_blk[RAPID3_MAX_NB];
    uint8_t u_flag[RAPID3_MAX_NB];
};

template <int D>
__host__ __device__ constexpr int tile_bytes() { return 128 * D * 2; }

template <int D>
constexpr size_t attn_smem_bytes() { return 3 * (size_t)tile_bytes<D>() + sizeof(Ctl) + 1024; }

template <int D>
__global__ void __launch_bounds__(NTHREADS, 2)
attn_kernel(const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
            const __grid_constant__ CUtensorMap tmv, const AttnParams prm) {
    constexpr int DH = D / 64;                 // 64-channel halves per row
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t pad = ((raw + 1023u) & ~1023u) - raw;
    uint8_t* smem = smem_raw + pad;
    const uint32_t sQ = raw + pad, sK = sQ + tile_bytes<D>(), sV = sK + tile_bytes<D>();
    Ctl* ctl = reinterpret_cast<Ctl*>(smem + 3 * tile_bytes<D>());

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int pair = blockIdx.x, h = blockIdx.y, p = blockIdx.z;
    const TensorGeom& g = prm.g;
    const int nb = g.nb, N = g.N;
    const int b = prm.imgs.batch[p], slot = prm.imgs.slot[p];
    const int i0 = 2 * pair;
    const bool has_q1 = (i0 + 1) < nb;

    uint32_t bar[N_BARS];
#pragma unroll
    for (int i = 0; i < N_BARS; ++i) bar[i] = smem_u32(&ctl->bars[i]);

    // ---------------------------------------------------------------- setup
    if (tid == 0) {
        mbar_init(bar[BAR_Q_FULL], 1);
        mbar_init(bar[BAR_K_FULL], 1);
        mbar_init(bar[BAR_K_EMPTY], 1);
        mbar_init(bar[BAR_V_FULL], 1);
        mbar_init(bar[BAR_V_EMPTY], 1);
        mbar_init(bar[BAR_S_FULL], 1);
        mbar_init(bar[BAR_P_FULL], 128);
        mbar_init(bar[BAR_PV_DONE], 1);
        ctl->abort_flag = 0;
        ctl->n_u = 0;
        fence_mbar_init();
        prefetch_tmap(&tmq);
        prefetch_tmap(&tmk);
        prefetch_tmap(&tmv);
    }
    if (tid < 64) ctl->bm[tid / 32][tid % 32] = 0;
    if (warp == 5) {
        tmem_alloc(smem_u32(&ctl->tmem_base), TMEM_COLS);
        tmem_relinquish();
        tc_fence_before();
    }
    __syncthreads();

    // ---------------------------------------------------------------- union of the two kept lists
    if (slot >= 0 && prm.kept_idx != nullptr) {
        for (int a = 0; a < (has_q1 ? 2 : 1); ++a) {
            const long long row = ((long long)slot * g.H + h) * nb + i0 + a;
            const int cnt = min(max(prm.kept_cnt[row], 0), nb);
            const int32_t* lst = prm.kept_idx + row * nb;
            for (int e = tid; e < cnt; e += NTHREADS) {
                const int j = lst[e];
                if ((unsigned)j < (unsigned)nb) atomicOr(&ctl->bm[a][j >> 5], 1u << (j & 31));
                else atomicExch(prm.status, RAPID3_ERR_BAD_LIST);
            }
        }
    } else if (tid < 32) {
        const int n = min(max(nb - tid * 32, 0), 32);
        const uint32_t val = n == 32 ? 0xffffffffu : ((1u << n) - 1u);
        ctl->bm[0][tid] = val;
        ctl->bm[1][tid] = has_q1 ? val : 0u;
    }
    __syncthreads();
    if (warp == 0) {
        const uint32_t m0 = ctl->bm[0][lane], m1 = ctl->bm[1][lane];
        uint32_t u = m0 | m1;
        const int c = __popc(u);
        int incl = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        int pos = incl - c;
        while (u) {
            const int bit = __ffs(u) - 1;
            u &= u - 1;
            ctl->u_blk[pos] = (int16_t)(lane * 32 + bit);
            ctl->u_flag[pos] = (uint8_t)(((m0 >> bit) & 1u) | (((m1 >> bit) & 1u) << 1));
            ++pos;
        }
        if (lane == 31) ctl->n_u = incl;
    }
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const int n_u = ctl->n_u;
    const int nt = (n_u + 1) / 2;

    auto fail = [&]() {
        atomicExch(prm.status, RAPID3_ERR_TIMEOUT);
        ctl->abort_flag = 1;
    };
    // bounded wait that also gives up quickly once another role has failed
    auto wait = [&](int which, uint32_t parity) -> bool {
        for (uint32_t it = 0; it < (1u << 22); ++it) {
            if (mbar_try_wait(bar[which], parity)) return true;
            if ((it & 255u) == 255u && ctl->abort_flag) return false;
        }
        fail();
        return false;
    };

    if (warp == 4) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            mbar_arrive_expect_tx(bar[BAR_Q_FULL], tile_bytes<D>());
#pragma unroll
            for (int c = 0; c < 2; ++c)
#pragma unroll
                for (int dh = 0; dh < DH; ++dh)
                    tma_load_4d(sQ + dh * HALF_BYTES + c * BLK_BYTES, &tmq, bar[BAR_Q_FULL], dh * 64, (i0 + c) * 64, h, b);
            int issued = 0;
            for (int t = 0; t < nt; ++t) {
                const int nblk = (2 * t + 1 < n_u) ? 2 : 1;
                const int j0 = ctl->u_blk[2 * t], j1 = nblk == 2 ? ctl->u_blk[2 * t + 1] : 0;
                if (!wait(BAR_K_EMPTY, (t & 1) ^ 1)) break;
                mbar_arrive_expect_tx(bar[BAR_K_FULL], nblk * 64 * D * 2);
                for (int c = 0; c < nblk; ++c)
#pragma unroll
                    for (int dh = 0; dh < DH; ++dh)
                        tma_load_4d(sK + dh * HALF_BYTES + c * BLK_BYTES, &tmk, bar[BAR_K_FULL], dh * 64,
                                    (c ? j1 : j0) * 64, h, b);
                if (!wait(BAR_V_EMPTY, (t & 1) ^ 1)) { issued = 2 * t + 1; break; }
                mbar_arrive_expect_tx(bar[BAR_V_FULL], nblk * 64 * D * 2);
                for (int c = 0; c < nblk; ++c)
#pragma unroll
                    for (int dh = 0; dh < DH; ++dh)
                        tma_load_4d(sV + dh * HALF_BYTES + c * BLK_BYTES, &tmv, bar[BAR_V_FULL], dh * 64,
                                    (c ? j1 : j0) * 64, h, b);
                issued = 2 * t + 2;
            }
            if (ctl->abort_flag) {
                // drain: do not leave the CTA while bulk copies may still land in its shared memory
                mbar_wait(bar[BAR_Q_FULL], 0, 1u << 20);
                if (issued >= 1) mbar_wait(bar[BAR_K_FULL], ((issued - 1) / 2) & 1, 1u << 20);
                if (issued >= 2) mbar_wait(bar[BAR_V_FULL], ((issued - 2) / 2) & 1, 1u << 20);
            }
        }
        __syncwarp();
    } else if (warp == 5) {
        // ------------------------------------------------------------ UMMA issue
        if (lane == 0) {
            const uint32_t tS = tmem_base + S_COL, tO = tmem_base + O_COL;
            constexpr uint32_t idesc_pv = idesc_bf16(128, D, 0, 1);
            bool ok = wait(BAR_Q_FULL, 0);
            for (int t = 0; ok && t < nt; ++t) {
                const int nkeys = (2 * t + 1 < n_u) ? 128 : 64;
                const uint32_t idesc_qk = idesc_bf16(128, nkeys, 0, 0);
                if (!(ok = wait(BAR_K_FULL, t & 1))) break;
                if (t > 0 && !(ok = wait(BAR_PV_DONE, (t - 1) & 1))) break;
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = (ks / 4) * HALF_BYTES + (ks % 4) * 32;
                    mma_ss(tS, smem_desc_sw128(sQ + off, 16, 1024), smem_desc_sw128(sK + off, 16, 1024), idesc_qk,
                           ks > 0);
                }
                tc_commit(bar[BAR_K_EMPTY]);
                tc_commit(bar[BAR_S_FULL]);
                if (!(ok = wait(BAR_P_FULL, t & 1))) break;
                if (!(ok = wait(BAR_V_FULL, t & 1))) break;
                tc_fence_after();
                for (int ks = 0; ks < nkeys / 16; ++ks)
                    mma_ts(tO, tS + ks * 8, smem_desc_sw128(sV + ks * 2048, HALF_BYTES, 1024), idesc_pv,
                           (t > 0 || ks > 0) ? 1u : 0u);
                tc_commit(bar[BAR_V_EMPTY]);
                tc_commit(bar[BAR_PV_DONE]);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ softmax / correction / epilogue
        const int a = warp >> 1;                       // which query block of the pair
        const int row = warp * 32 + lane;              // row of the 128-row tile == TMEM lane
        const uint32_t lane_addr = tmem_base + ((uint32_t)(warp * 32) << 16);
        const uint32_t tS = lane_addr + S_COL, tO = lane_addr + O_COL;
        const float c2 = prm.scale_log2;
        const int tail_valid = N - (nb - 1) * 64;      // valid tokens of the last block (1..64)
        float m_run = -INFINITY, l_run = 0.f;
        bool ok = true;
        uint32_t r[32];
        for (int t = 0; t < nt; ++t) {
            const int nhalf = (2 * t + 1 < n_u) ? 2 : 1;
            bool act[2];
            int valid[2];
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const bool have = c < nhalf;
                const int j = have ? ctl->u_blk[2 * t + c] : 0;
                act[c] = have && ((ctl->u_flag[2 * t + c] >> a) & 1);
                valid[c] = (j == nb - 1) ? tail_valid : 64;
            }
            if (!(ok = wait(BAR_S_FULL, t & 1))) break;
            tc_fence_after();
            // pass 1: row maximum over the active, valid columns
            float mx = -INFINITY;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                if (!act[c]) continue;
#pragma unroll
                for (int qd = 0; qd < 2; ++qd) {
                    tmem_ld32(tS + c * 64 + qd * 32, r);
                    tc_wait_ld();
                    if (valid[c] == 64) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) mx = fmaxf(mx, __uint_as_float(r[e]));
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (qd * 32 + e < valid[c]) mx = fmaxf(mx, __uint_as_float(r[e]));
                    }
                }
            }
            // lazy rescale: move the reference maximum only when it grew by more than 2^8
            const float m_new = fmaxf(m_run, mx);
            const bool grow = (m_new > m_run) && ((m_new - m_run) * c2 > RESCALE_LOG2);
            if (t > 0 && __any_sync(0xffffffffu, grow)) {
                const float alpha = grow ? ex2((m_run - m_new) * c2) : 1.f;
                l_run *= alpha;
#pragma unroll
                for (int ch = 0; ch < D / 32; ++ch) {
                    tmem_ld32(tO + ch * 32, r);
                    tc_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
                    tmem_st32(tO + ch * 32, r);
                }
            }
            if (grow) m_run = m_new;
            const float ms = m_run * c2;
            // pass 2: P = exp2(S * c2 - ms), row sum, bf16 P over the consumed S columns
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                if (c >= nhalf) continue;
#pragma unroll
                for (int qd = 0; qd < 2; ++qd) {
                    uint32_t pk[16];
                    if (act[c]) {
                        tmem_ld32(tS + c * 64 + qd * 32, r);
                        tc_wait_ld();
                        float pv[32];
#pragma unroll
                        for (int e = 0; e < 32; ++e) {
                            float x = ex2(fmaf(__uint_as_float(r[e]), c2, -ms));
                            if (valid[c] != 64 && qd * 32 + e >= valid[c]) x = 0.f;
                            pv[e] = x;
                            l_run += x;
                        }
#pragma unroll
                        for (int e = 0; e < 16; ++e) pk[e] = pack_bf16(pv[2 * e], pv[2 * e + 1]);
                    } else {
#pragma unroll
                        for (int e = 0; e < 16; ++e) pk[e] = 0u;
                    }
                    tmem_st16(tS + c * 32 + qd * 16, pk);
                }
            }
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(bar[BAR_P_FULL]);
        }
        // epilogue: O / l -> bf16 -> global
        const int n_glob = i0 * 64 + row;
        uint16_t* orow = prm.out + (long long)b * g.stride_b + (long long)h * g.stride_h + (long long)n_glob * g.stride_n;
        if (ok && nt > 0) ok = wait(BAR_PV_DONE, (nt - 1) & 1);
        if (ok) {
            tc_fence_after();
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
#pragma unroll
            for (int ch = 0; ch < D / 32; ++ch) {
                if (nt > 0) {
                    tmem_ld32(tO + ch * 32, r);
                    tc_wait_ld();
                } else {
#pragma unroll
                    for (int e = 0; e < 32; ++e) r[e] = 0u;
                }
                if (n_glob < N) {
#pragma unroll
                    for (int v4 = 0; v4 < 4; ++v4) {
                        uint4 o;
                        o.x = pack_bf16(__uint_as_float(r[v4 * 8 + 0]) * inv, __uint_as_float(r[v4 * 8 + 1]) * inv);
                        o.y = pack_bf16(__uint_as_float(r[v4 * 8 + 2]) * inv, __uint_as_float(r[v4 * 8 + 3]) * inv);
                        o.z = pack_bf16(__uint_as_float(r[v4 * 8 + 4]) * inv, __uint_as_float(r[v4 * 8 + 5]) * inv);
                        o.w = pack_bf16(__uint_as_float(r[v4 * 8 + 6]) * inv, __uint_as_float(r[v4 * 8 + 7]) * inv);
                        *reinterpret_cast<uint4*>(orow + ch * 32 + v4 * 8) = o;
                    }
                }
            }
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        if (ctl->abort_flag && lane == 0) {
            // make sure no UMMA is still in flight before the TMEM columns are released
            tc_commit(bar[BAR_Q_FULL]);
            mbar_wait(bar[BAR_Q_FULL], 1, 1u << 20);
        }
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

bool g_attr_set = false;

}  // namespace

cudaError_t attention_static_init() {
    cudaError_t e = cudaFuncSetAttribute(attn_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)attn_smem_bytes<128>());
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_smem_bytes<64>());
    if (e != cudaSuccess) return e;
    g_attr_set = true;
    return cudaSuccess;
}

cudaError_t launch_attention(const CUtensorMap& tmq, const CUtensorMap& tmk, const CUtensorMap& tmv, void* out,
                             const TensorGeom& g, const ImgList& imgs, const int32_t* kept_idx,
                             const int32_t* kept_cnt, float softmax_scale, int* status, cudaStream_t s) {
    if (!g_attr_set) {
        cudaError_t e = attention_static_init();
        if (e != cudaSuccess) return e;
    }
    AttnParams prm;
    prm.g = g;
    prm.imgs = imgs;
    prm.kept_idx = kept_idx;
    prm.kept_cnt = kept_cnt;
    prm.out = reinterpret_cast<uint16_t*>(out);
    prm.status = status;
    prm.scale_log2 = softmax_scale * 1.4426950408889634f;
    dim3 grid((g.nb + 1) / 2, g.H, imgs.n);
    if (g.D == 128)
        attn_kernel<128><<<grid, NTHREADS, attn_smem_bytes<128>(), s>>>(tmq, tmk, tmv, prm);
    else
        attn_kernel<64><<<grid, NTHREADS, attn_smem_bytes<64>(), s>>>(tmq, tmk, tmv, prm);
    return cudaGetLastError();
}
