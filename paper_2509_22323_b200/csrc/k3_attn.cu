// K3: masked flash-style joint attention over the kept key tiles (sm_100a).
//
// One CTA per (image, head, four adjacent 64-token query blocks) = two 128-row Q tiles (the
// native UMMA M), one CTA per SM.  The four query blocks' ascending kept lists are merged into
// one union list; the producer streams each key block of the union once through shared memory
// and both tiles use it, which nearly halves the L2 -> SM traffic per MMA and leaves room for
// deep K / V rings.  A tile issues no MMA for a key block that neither of its query blocks
// kept; inside a tile a 64x64 sub-tile whose key block is not in that query block's own list
// gets P = 0, so each query block attends exactly its own kept set.
//
// Roles (608 threads):
//   warp 16     producer: TMA loads (cp.async.bulk.tensor, 128-byte swizzle) of Q once, then
//               the gathered K and V blocks into two rings of shared-memory stages; K(g) and
//               V(g - 1), which the MMA warps need together, complete one barrier
//   warps 17,18 UMMA issue, one warp per tile (warp 17 also owns the TMEM allocation).  S of a
//               tile has NBUF buffers in TMEM (64 fp32 columns each): S(n + NBUF - 1) = Q K^T is
//               issued before O += P(n) V, so the tensor pipe works on the next scores while the
//               softmax warps are busy with the current ones.  Both warps walk the same union
//               list, K ahead of V; a stage is released when both have passed it
//   warps 0-15  softmax, eight warps per tile and four per SM sub-partition: a warp owns 16 query rows, a
//               thread a quarter of two rows (16x256b fragments; 32 scores per key block); fp32 online
//               softmax with lazy rescale of O, P(n) written back over S(n) as bf16, final O / l store
// TMEM: tile t owns columns [256 t, 256 t + 256): S(n) at 64 (n mod NBUF), O behind the NBUF score buffers
// (two of them and O at 128 for D = 128; three and O at 192 for D = 64, where the columns allow it).
// Every mbarrier wait is bounded; a wait that runs out records RAPID3_ERR_TIMEOUT in the status
// word and the CTA drains its copies, releases its TMEM and exits normally.
#include "common.cuh"
#include "ptx.cuh"

using namespace ptx;

// score buffers per tile: three where the TMEM columns allow it (D = 64: 3 x 64 + 64 of O), else two
#define RAPID3_NBUF(D) ((D) == 64 ? 3 : 2)
namespace {

constexpr int SOFTMAX_WARPS = 16;
constexpr int PRODUCER_WARP = 16, MMA_WARP0 = 17;
constexpr int NTHREADS = 32 * (SOFTMAX_WARPS + 3);
constexpr int TMEM_COLS = 512;
constexpr int TILE_COLS = 256;      // TMEM columns of one Q tile
constexpr int BLK_BYTES = 8192;     // 64 rows x 128 bytes: one 64-channel half of a 64-token block
constexpr int QHALF_BYTES = 16384;  // one 64-channel half of a 128-row Q tile
constexpr float RESCALE_LOG2 = 8.0f;
constexpr int MAX_STAGES = 8;

struct AttnParams {
    TensorGeom g;
    ImgList imgs;
    const int32_t* kept_idx;
    const int32_t* kept_cnt;
    const uint32_t* bitmask32;     // optional: the same mask as 32-bit words, [slot][H][nb][words32]
    int words32;
    int n_dense;                   // leading images of the list that keep every block
    const DevPlan* plan;           // optional: image list and n_dense from device memory (grid sized for n_cap images)
    int* status;
    float scale_log2;
    int stop_group;                // failure-injection build of the kernel only: the producer stops before this group
};

template <int D>
struct Cfg {
    static constexpr int DH = D / 64;                       // 64-channel halves per row
    static constexpr int QTILE_BYTES = 128 * D * 2;         // one 128-row Q tile
    static constexpr int KV_BYTES = 64 * D * 2;             // one key block of K or of V
    static constexpr int KS = (D == 128) ? 4 : 8;           // K ring stages
    static constexpr int VS = (D == 128) ? 4 : 8;           // V ring stages
    static constexpr int DATA_BYTES = 2 * QTILE_BYTES + (KS + VS) * KV_BYTES;
    static constexpr int NBUF = RAPID3_NBUF(D);             // score buffers (64 columns each) per tile
    static constexpr int O_COL = 64 * NBUF;                 // O accumulator behind them: 64 NBUF + D <= 256 columns per tile
};

struct __align__(16) Ctl {
    unsigned long long q_full;
    unsigned long long k_full[MAX_STAGES], k_empty[MAX_STAGES];   // k_full[g % KS]: group g = K(g) and V(g - 1) have landed
    unsigned long long v_empty[MAX_STAGES];
    unsigned long long s_full[2][3], p_full[2][3];
    unsigned long long pv_done[2][2], o_done[2], drain[2];
    uint32_t tmem_base;
    int n_u;
    volatile int abort_flag;
    uint32_t bm[4][32];
    int16_t u_blk[RAPID3_MAX_NB];
    uint8_t u_flag[RAPID3_MAX_NB];      // bit a: query block a of the quad keeps this key block
};

template <int D>
constexpr size_t attn_smem_bytes() { return (size_t)Cfg<D>::DATA_BYTES + sizeof(Ctl) + 1024; }

__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// INJECT = true is the failure-injection build behind rapid3_debug_inject_timeout: the producer
// stops before group prm.stop_group and every wait gives up after 2^12 polls, so the waits of all
// roles run out and the abort path (status word, drain of the copies in flight, UMMA drain, TMEM
// release) is what runs.  The product launches only use INJECT = false.
template <int D, bool INJECT = false>
__global__ void __launch_bounds__(NTHREADS, 1)
attn_kernel(const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
            const __grid_constant__ CUtensorMap tmv, const __grid_constant__ CUtensorMap tmo, const AttnParams prm) {
    using C = Cfg<D>;
    constexpr int DH = C::DH, KS = C::KS, VS = C::VS, NBUF = C::NBUF, O_COL = C::O_COL;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t pad = ((raw + 1023u) & ~1023u) - raw;
    uint8_t* smem = smem_raw + pad;
    const uint32_t sQ = raw + pad, sK = sQ + 2 * C::QTILE_BYTES, sV = sK + KS * C::KV_BYTES;
    Ctl* ctl = reinterpret_cast<Ctl*>(smem + C::DATA_BYTES);

    const int tid = threadIdx.x, lane = tid % 32;
    // the shuffle makes the warp index provably warp-uniform, so role branches and the address
    // arithmetic inside them can live in uniform registers
    const int warp = __shfl_sync(0xffffffffu, tid / 32, 0);
    const TensorGeom& g = prm.g;
    const int nb = g.nb, N = g.N;
    // Work order, longest first (CTAs start in block-index order as SMs free up, so this is
    // longest-processing-time-first scheduling): every quad of the dense images and the quads of
    // the sparse images that hold a text query block walk all nb key blocks; the other quads of the
    // sparse images follow, image by image in the list's order (descending keep ratio).
    int quad, h, p, b, slot;
    {
        const int nq = (nb + 3) >> 2, ntq = min(nq, (g.n_text_blocks + 3) >> 2);
        const int n_all = prm.plan ? prm.plan->all.n : prm.imgs.n;
        const int nd = prm.plan ? prm.plan->n_dense : prm.n_dense, ns = n_all - nd;
        int L = blockIdx.x;
        if (L >= nq * g.H * n_all) return;               // device-resident plan: fewer images than the grid covers
        const int heavy_dense = nd * g.H * nq, heavy_sparse = ns * g.H * ntq;
        if (L < heavy_dense) {
            p = L / (g.H * nq); L -= p * g.H * nq;
            h = L / nq; quad = L - h * nq;
        } else if (L < heavy_dense + heavy_sparse) {
            L -= heavy_dense;
            p = L / (g.H * ntq); L -= p * g.H * ntq; p += nd;
            h = L / ntq; quad = L - h * ntq;
        } else {
            L -= heavy_dense + heavy_sparse;
            const int nl = nq - ntq;
            p = L / (g.H * nl); L -= p * g.H * nl; p += nd;
            h = L / nl; quad = ntq + (L - h * nl);
        }
        b = prm.plan ? prm.plan->all.batch[p] : prm.imgs.batch[p];
        slot = prm.plan ? prm.plan->all.slot[p] : prm.imgs.slot[p];
    }
    const int i0 = 4 * quad;
    // Which two of the quad's four query blocks form a 128-row tile: neighbours (a, a + 1), or, when
    // a row of the image grid spans two blocks, vertical neighbours (a, a + 2), whose kept lists
    // overlap far more (measured on the 128 x 128 grid at keep ratio 0.25: 90 % against 63 % of
    // the tile's MMA work lands on kept 64 x 64 sub-tiles).
    // pair_stride 3 goes further on that grid: the whole quad is one column of it -- members
    // (b, b + 2, b + 4, b + 6), the left or the right halves of four consecutive grid rows -- so both
    // tiles want nearly the same key blocks (union of the quad 98 instead of 134 blocks at keep ratio
    // 0.25, both tiles busy on 68 % of them instead of 23 %).  qblk(a) is member a's query block.
    const bool ps2 = g.pair_stride == 2;
    const bool vq = g.pair_stride == 3;
    auto qblk = [&](int a) -> int {
        int i = i0 + a;
        if (vq && i >= g.n_text_blocks) {
            const int r = i - g.n_text_blocks, w = r & 7;
            i = g.n_text_blocks + (r & ~7) + ((w & 3) << 1) + (w >> 2);
        }
        return i;
    };

    const uint32_t bQ = smem_u32(&ctl->q_full);
    const uint32_t bKF = smem_u32(&ctl->k_full[0]), bKE = smem_u32(&ctl->k_empty[0]);
    const uint32_t bVE = smem_u32(&ctl->v_empty[0]);
    const uint32_t bSF = smem_u32(&ctl->s_full[0][0]), bPF = smem_u32(&ctl->p_full[0][0]);   // [tile][buf]: + 24 t + 8 buf
    const uint32_t bPV = smem_u32(&ctl->pv_done[0][0]);                                      // [tile][block parity]: + 16 t + 8 (n & 1)
    const uint32_t bOD = smem_u32(&ctl->o_done[0]);                                          // [tile]: + 8 t

    // ---------------------------------------------------------------- setup
    if (warp == 0) {                                    // one barrier group per lane
        if (lane < MAX_STAGES) {
            mbar_init(bKF + 8 * lane, 1);
            mbar_init(bKE + 8 * lane, 2);   // both tiles pass a stage before it is refilled
            mbar_init(bVE + 8 * lane, 2);
        } else if (lane < MAX_STAGES + 6) {
            mbar_init(bSF + 8 * (lane - MAX_STAGES), 1);
            mbar_init(bPF + 8 * (lane - MAX_STAGES), 8);      // one arrival per softmax warp of the tile
        } else if (lane < MAX_STAGES + 8) {
            const int t = lane - MAX_STAGES - 6;
            mbar_init(bPV + 16 * t, 1);
            mbar_init(bPV + 16 * t + 8, 1);
            mbar_init(bOD + 8 * t, 1);
            mbar_init(smem_u32(&ctl->drain[t]), 1);
        } else if (lane == MAX_STAGES + 8) {
            mbar_init(bQ, 1);
            ctl->abort_flag = 0;
            ctl->n_u = 0;
        } else if (lane == MAX_STAGES + 9) {
            prefetch_tmap(&tmq);
            prefetch_tmap(&tmk);
            prefetch_tmap(&tmv);
            prefetch_tmap(&tmo);
        }
        fence_mbar_init();
    }
    if (tid < 128) ctl->bm[tid / 32][tid % 32] = 0;
    if (warp == MMA_WARP0) {
        tmem_alloc(smem_u32(&ctl->tmem_base), TMEM_COLS);
        tmem_relinquish();
        tc_fence_before();
    }
    __syncthreads();

    // Key blocks known before the mask is read: a dense image keeps every block, and a mask of the selection kernel
    // keeps the text blocks in every row, so the union list starts 0, 1, ... -- their K (and V) loads can start now.
    const int n_early = (!INJECT && (slot < 0 || prm.bitmask32 != nullptr)) ? min(min(slot < 0 ? nb : g.n_text_blocks, nb), KS) : 0;
    // The Q tiles do not depend on the mask: start their loads before the union list is built.
    if (warp == PRODUCER_WARP && lane == 0) {
        mbar_arrive_expect_tx(bQ, 2 * C::QTILE_BYTES);
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int dh = 0; dh < DH; ++dh)
                tma_load_4d(sQ + (ps2 ? (a & 1) : (a >> 1)) * C::QTILE_BYTES + dh * QHALF_BYTES +
                                (ps2 ? (a >> 1) : (a & 1)) * BLK_BYTES, &tmq, bQ,
                            dh * 64, qblk(a) * 64, g.h0 + h, b);
        // groups 0 .. n_early - 1 (group g = K(g) with V(g - 1)): first use of their stages, nothing to wait for
        for (int gi = 0; gi < n_early; ++gi) {
            mbar_arrive_expect_tx(bKF + 8 * gi, C::KV_BYTES + (gi > 0 ? C::KV_BYTES : 0));
#pragma unroll
            for (int dh = 0; dh < DH; ++dh)
                tma_load_4d(sK + gi * C::KV_BYTES + dh * BLK_BYTES, &tmk, bKF + 8 * gi, dh * 64, gi * 64, g.h0 + h, b);
            if (gi > 0) {
#pragma unroll
                for (int dh = 0; dh < DH; ++dh)
                    tma_load_4d(sV + (gi - 1) * C::KV_BYTES + dh * BLK_BYTES, &tmv, bKF + 8 * gi, dh * 64, (gi - 1) * 64, g.h0 + h, b);
            }
        }
    }

    // ---------------------------------------------------------------- union of the four kept lists
    // bm[a] = bit set of the key blocks query block a keeps: copied from the bitmask when the
    // caller has one, else rebuilt from the kept list; every block is kept for a dense image.
    const int nw = (nb + 31) >> 5;
    // Launched as a dependent of the selection kernel, a thread block of a sparse image waits here for the masks; one of
    // a dense image reads nothing of them and runs on (an idle lane of its producer warp waits instead, so that the
    // grid as a whole still ends after the selection kernel).  The masks are read past the L1 (ld.global.cg): this thread block may have
    // started before they were written, and an L1 line of an earlier step must not answer.
    if (slot >= 0) grid_dependency_wait();
    if (slot >= 0 && prm.bitmask32 != nullptr) {
        if (tid < 4 * nw) {
            const int a = tid / nw, w = tid - a * nw;
            if (qblk(a) < nb)
                ctl->bm[a][w] = __ldcg(prm.bitmask32 + (((long long)slot * g.H + h) * nb + qblk(a)) * prm.words32 + w);
        }
    } else if (slot >= 0 && prm.kept_idx != nullptr) {
        for (int a = 0; a < 4 && qblk(a) < nb; ++a) {
            const long long row = ((long long)slot * g.H + h) * nb + qblk(a);
            const int cnt = min(max(__ldcg(prm.kept_cnt + row), 0), nb);
            const int32_t* lst = prm.kept_idx + row * nb;
            for (int e = tid; e < cnt; e += NTHREADS) {
                const int j = __ldcg(lst + e);
                if ((unsigned)j < (unsigned)nb) atomicOr(&ctl->bm[a][j >> 5], 1u << (j & 31));
                else atomicExch(prm.status, RAPID3_ERR_BAD_LIST);
            }
        }
    } else if (tid < 32) {
        const int n = min(max(nb - tid * 32, 0), 32);
        const uint32_t val = n == 32 ? 0xffffffffu : ((1u << n) - 1u);
        for (int a = 0; a < 4; ++a) ctl->bm[a][tid] = (qblk(a) < nb) ? val : 0u;
    }
    __syncthreads();
    // one thread per key block: its position in the ascending union list is the number of union
    // bits below it
    for (int j = tid; j < nb; j += NTHREADS) {
        const int w = j >> 5, bit = j & 31;
        const uint32_t m0 = ctl->bm[0][w], m1 = ctl->bm[1][w], m2 = ctl->bm[2][w], m3 = ctl->bm[3][w];
        const uint32_t u = m0 | m1 | m2 | m3;
        if ((u >> bit) & 1u) {
            int pos = __popc(u & ((1u << bit) - 1u));
            for (int x = 0; x < w; ++x) pos += __popc(ctl->bm[0][x] | ctl->bm[1][x] | ctl->bm[2][x] | ctl->bm[3][x]);
            ctl->u_blk[pos] = (int16_t)j;
            ctl->u_flag[pos] = (uint8_t)(((m0 >> bit) & 1u) | (((m1 >> bit) & 1u) << 1) | (((m2 >> bit) & 1u) << 2) |
                                         (((m3 >> bit) & 1u) << 3));
        }
    }
    if (tid == 0) {
        int tot = 0;
        for (int x = 0; x < nw; ++x) tot += __popc(ctl->bm[0][x] | ctl->bm[1][x] | ctl->bm[2][x] | ctl->bm[3][x]);
        ctl->n_u = tot;
    }
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const int n_u = ctl->n_u;

    auto fail = [&]() {
        atomicExch(prm.status, RAPID3_ERR_TIMEOUT);
        ctl->abort_flag = 1;
    };
    // bounded wait that also gives up quickly once another role has failed
    auto wait = [&](uint32_t bar, uint32_t parity) -> bool {
        constexpr uint32_t limit = INJECT ? (1u << 12) : (1u << 22);
        for (uint32_t it = 0; it < limit; ++it) {
            if (mbar_try_wait(bar, parity)) return true;
            if ((it & 255u) == 255u && ctl->abort_flag) return false;
        }
        fail();
        return false;
    };
    // the same for a converged warp, with a warp-uniform result
    auto wait_warp = [&](uint32_t bar, uint32_t parity) -> bool {
        return __all_sync(0xffffffffu, wait(bar, parity));
    };

    if (warp == PRODUCER_WARP) {
        // ------------------------------------------------------------ producer
        if (slot < 0 && lane == 1) grid_dependency_wait();   // see above; off every critical path
        if (lane == 0) {
            // Group g = K block g together with V block g - 1: the MMA warps need exactly that pair before they
            // issue S(g) = Q K(g)^T and O += P(g-1) V(g-1), so the pair completes ONE barrier (g_full[g % KS]) and
            // costs them one wait per key block instead of two.  Group 0 is K(0) alone, group n_u is V(n_u - 1)
            // alone.  A group is armed once both ring stages it fills have been released.
            int g_issued = n_early;
            auto load_group = [&](int gi) -> bool {
                const int s = gi % KS;
                const bool has_k = gi < n_u, has_v = gi > 0;
                // the K stage's release also tells that both MMA warps are past their wait on this barrier's
                // previous phase (group gi - KS), so it is awaited even when group n_u brings no K block
                if (!wait(bKE + 8 * s, ((gi / KS) & 1) ^ 1)) return false;
                const int jv = gi - 1, sv = has_v ? jv % VS : 0;
                if (has_v && !wait(bVE + 8 * sv, ((jv / VS) & 1) ^ 1)) return false;
                mbar_arrive_expect_tx(bKF + 8 * s, (has_k ? C::KV_BYTES : 0) + (has_v ? C::KV_BYTES : 0));
                if (has_k) {
                    const int blk = ctl->u_blk[gi];
#pragma unroll
                    for (int dh = 0; dh < DH; ++dh)
                        tma_load_4d(sK + s * C::KV_BYTES + dh * BLK_BYTES, &tmk, bKF + 8 * s, dh * 64, blk * 64, g.h0 + h, b);
                }
                if (has_v) {
                    const int blk = ctl->u_blk[jv];
#pragma unroll
                    for (int dh = 0; dh < DH; ++dh)
                        tma_load_4d(sV + sv * C::KV_BYTES + dh * BLK_BYTES, &tmv, bKF + 8 * s, dh * 64, blk * 64, g.h0 + h, b);
                }
                g_issued = gi + 1;
                return true;
            };
            bool ok = true;
            for (int gi = n_early; ok && n_u > 0 && gi <= n_u; ++gi) {
                if (INJECT && gi == prm.stop_group) break;
                ok = load_group(gi);
            }
            if (INJECT || ctl->abort_flag) {
                // drain: do not leave the CTA while bulk copies may still land in its shared memory
                mbar_wait(bQ, 0, 1u << 20);
                for (int gi = max(0, g_issued - KS); gi < g_issued; ++gi)
                    mbar_wait(bKF + 8 * (gi % KS), (gi / KS) & 1, 1u << 20);
            }
        }
        __syncwarp();
    } else if (warp >= MMA_WARP0) {
        // ------------------------------------------------------------ UMMA issue, one warp per tile
        // At D = 128 the whole warp runs the loop converged (addresses and descriptors stay warp-uniform) and
        // one elected lane issues the tcgen05 instructions; at D = 64, where the time between a barrier's
        // completion and the next issue shows in the launch time, the elected lane runs the loop alone, without
        // the votes and warp barriers that convergence costs (measured: 1.8 % faster at D = 64, 0.4 % slower at
        // D = 128).  Both warps pass over every block of
        // the union list, K one block ahead of V, also over blocks their tile does not use: the
        // stage barriers then see every phase in order and a stage is refilled only after both
        // tiles are past it.
        const int t = warp - MMA_WARP0;
        const uint32_t tile_bits = ps2 ? (5u << t) : (3u << (2 * t));
        constexpr bool SOLO = (D == 64);
        const bool leader = elect_one();
        auto mma_wait = [&](uint32_t bar, uint32_t parity) -> bool {
            if constexpr (SOLO) return wait(bar, parity);
            else return wait_warp(bar, parity);
        };
        if (!SOLO || leader) {
            const uint32_t tbase = tmem_base + t * TILE_COLS;
            const uint32_t tO = tbase + O_COL;
            const uint32_t qb = sQ + t * C::QTILE_BYTES;
            const uint32_t bSFt = bSF + 24 * t, bPFt = bPF + 24 * t;
            constexpr uint32_t idesc_qk = idesc_bf16(128, 64, 0, 0);
            constexpr uint32_t idesc_pv = idesc_bf16(128, D, 0, 1);
            int n_qk = 0, n_pv = 0;                        // blocks of this tile issued so far
            // waits for group gi (K(gi) and V(gi - 1), see the producer), then issues S = Q K(gi)^T
            auto k_step = [&](int j) -> bool {
                const int s = j % KS;
                if (!(mma_wait(bKF + 8 * s, (j / KS) & 1))) return false;
                if (j >= n_u) return true;                 // the last group holds V(n_u - 1) only
                const bool use = ctl->u_flag[j] & tile_bits;
                if (use) {
                    tc_fence_after();
                    const uint32_t tS = tbase + 64 * (n_qk % NBUF);
                    const uint32_t kb = sK + s * C::KV_BYTES;
                    if (leader) {
    #pragma unroll
                        for (int ks = 0; ks < D / 16; ++ks)
                            mma_ss(tS, smem_desc_sw128(qb + (ks / 4) * QHALF_BYTES + (ks % 4) * 32, 16, 1024),
                                   smem_desc_sw128(kb + (ks / 4) * BLK_BYTES + (ks % 4) * 32, 16, 1024), idesc_qk, ks > 0);
                        tc_commit(bKE + 8 * s);
                        tc_commit(bSFt + 8 * (n_qk % NBUF));
                    }
                    ++n_qk;
                } else if (leader) {
                    mbar_arrive(bKE + 8 * s);
                }
                if (!SOLO) __syncwarp();
                return true;
            };
            bool ok = (mma_wait(bQ, 0));
            // the scores run NBUF - 1 key blocks ahead of the P V products
            for (int j = 0; ok && j < NBUF - 1 && j <= n_u && n_u > 0; ++j) ok = k_step(j);
            for (int j = 0; ok && j < n_u; ++j) {
                // S(n + NBUF - 1) reuses the buffer of P(n - 1); the MMAs of the issuing thread execute in issue
                // order, so it is written only after P(n - 1) V has read it
                if (j + NBUF - 1 <= n_u && !(ok = k_step(j + NBUF - 1))) break;          // group j + 1 brings V(j)
                const int s = j % VS;
                const bool use = ctl->u_flag[j] & tile_bits;
                if (use && !(ok = (mma_wait(bPFt + 8 * (n_pv % NBUF), (n_pv / NBUF) & 1)))) break;
                if (use) {
                    tc_fence_after();
                    const uint32_t tP = tbase + 64 * (n_pv % NBUF);
                    const uint32_t vb = sV + s * C::KV_BYTES;
                    if (leader) {
    #pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            mma_ts(tO, tP + ks * 8, smem_desc_sw128(vb + ks * 2048, BLK_BYTES, 1024), idesc_pv,
                                   (n_pv > 0 || ks > 0) ? 1u : 0u);
                        tc_commit(bVE + 8 * s);
                        // pv_done: two barriers per tile, for the even and the odd blocks.  The softmax warps run up
                        // to NBUF - 1 <= 2 blocks ahead of these products, and the parity of one barrier taking every
                        // block could not tell "block n - 1 is done" from "block n - 3 is done"; with two, the one the
                        // rescale path waits on (block n - 1's) can only be one phase behind, because S(n) exists only
                        // once the product of block n - NBUF is over.  The epilogue may lag, so it has its own barrier.
                        tc_commit(bPV + 16 * t + 8 * (n_pv & 1));
                    }
                    ++n_pv;
                } else if (leader) {
                    mbar_arrive(bVE + 8 * s);
                }
                if (!SOLO) __syncwarp();
            }
            if (ok && leader && n_pv > 0) tc_commit(bOD + 8 * t);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ softmax / correction / epilogue
        // Sixteen warps, four per SM sub-partition, so that while one waits on a barrier or on tensor memory
        // the others keep the exponential unit busy.  Warp w works on tile (w >> 2) & 1, on the 16 rows
        // 32 (w & 3) + 16 (w >> 3) .. + 15 of it, with the 16x256b fragment layout: a thread owns two rows
        // (r_lo = lane / 4 and r_lo + 8 of the sixteen) and, of every group of eight score columns, the pair
        // 2 (lane % 4), + 1 -- 32 scores per key block.  The four threads of a quad share their rows' maximum
        // with two shuffles, and only when some row of the warp may have grown.
        const int t = (warp >> 2) & 1, wl = warp & 3, hf = warp >> 3;
        const int a = ps2 ? 2 * (wl >> 1) + t : 2 * t + (wl >> 1);   // query block of the quad
        const uint32_t tile_bits = ps2 ? (5u << t) : (3u << (2 * t));
        const int cg = lane & 3;                        // column pair within a group of eight
        const int row_lo = wl * 32 + hf * 16 + (lane >> 2);          // row of the 128-row tile; the second row is + 8
        const uint32_t lane_addr = tmem_base + ((uint32_t)(wl * 32 + hf * 16) << 16) + t * TILE_COLS;
        const uint32_t tO = lane_addr + O_COL;
        const uint32_t bSFt = bSF + 24 * t, bPFt = bPF + 24 * t, bPVt = bPV + 16 * t;
        const float c2 = prm.scale_log2;
        const int tail_valid = N - (nb - 1) * 64;      // valid tokens of the last block (1..64)
        float m_lo = -INFINITY, m_hi = -INFINITY;      // reference maxima of the two rows
        float l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;  // partial row sums: (l0, l1) first row, (l2, l3) second row
        bool ok = true;
        uint32_t r[32];
        int n = 0;                                     // blocks of this tile so far
        bool seeded = false;                           // the rows' reference maxima have been set (warp-uniform: a warp's rows share a query block)
        for (int j = 0; j < n_u; ++j) {
            const uint32_t f = ctl->u_flag[j];
            if (!(f & tile_bits)) continue;            // neither query block of the tile kept it
            const int blk = ctl->u_blk[j];
            const bool act = (f >> a) & 1u;
            const int valid = (blk == nb - 1) ? tail_valid : 64;
            const int buf = n % NBUF;
            const uint32_t tS = lane_addr + 64 * buf;
            if (!(ok = wait_warp(bSFt + 8 * buf, (n / NBUF) & 1))) break;
            tc_fence_after();
            uint32_t pk[16];
            if (act) {
                tmem_ld16x256_x8(tS, r);
                tc_wait_ld();
                if (valid != 64) {
#pragma unroll
                    for (int k = 0; k < 8; ++k)
#pragma unroll
                        for (int e = 0; e < 2; ++e)
                            if (8 * k + 2 * cg + e >= valid) {       // -inf: outside the sequence
                                r[4 * k + e] = 0xff800000u;
                                r[4 * k + 2 + e] = 0xff800000u;
                            }
                }
                // One pass over the 32 scores gives P = 2^(S c2 - m c2) (packed to bf16), the block's partial
                // row sums and the thread's share of the block's row maxima.  The pass runs with the reference
                // maxima as they stand, so the exponentials do not wait for this block's maximum; only when a
                // row's maximum has grown by more than 2^8 (rare after the first blocks) O and l are rescaled
                // and the pass is repeated.
                float b0, b1, b2, b3;
                bool redo;
                if (!seeded) {
                    // the first block this query block keeps: take the rows' maxima before the pass instead of running
                    // the pass twice (from -inf every row "grows")
                    float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        mx_lo = max3(mx_lo, __uint_as_float(r[4 * k]), __uint_as_float(r[4 * k + 1]));
                        mx_hi = max3(mx_hi, __uint_as_float(r[4 * k + 2]), __uint_as_float(r[4 * k + 3]));
                    }
                    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
                    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
                    m_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
                    m_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
                    seeded = true;
                }
                do {
                    const float ms_lo = m_lo * c2, ms_hi = m_hi * c2;
                    float mx_lo = -INFINITY, mx_hi = -INFINITY;
                    b0 = b1 = b2 = b3 = 0.f;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        float x0, x1, x2, x3;
                        fma2(x0, x1, __uint_as_float(r[4 * k]), __uint_as_float(r[4 * k + 1]), c2, -ms_lo);
                        fma2(x2, x3, __uint_as_float(r[4 * k + 2]), __uint_as_float(r[4 * k + 3]), c2, -ms_hi);
                        x0 = ex2(x0); x1 = ex2(x1); x2 = ex2(x2); x3 = ex2(x3);
                        add2(b0, b1, x0, x1);
                        add2(b2, b3, x2, x3);
                        pk[2 * k] = pack_bf16(x0, x1);
                        pk[2 * k + 1] = pack_bf16(x2, x3);
                        mx_lo = max3(mx_lo, __uint_as_float(r[4 * k]), __uint_as_float(r[4 * k + 1]));
                        mx_hi = max3(mx_hi, __uint_as_float(r[4 * k + 2]), __uint_as_float(r[4 * k + 3]));
                    }
                    // a thread sees a quarter of each row: if any thread of the warp sees growth, the quads
                    // combine their maxima and decide row by row
                    redo = __any_sync(0xffffffffu, (mx_lo - m_lo) * c2 > RESCALE_LOG2 || (mx_hi - m_hi) * c2 > RESCALE_LOG2);
                    if (redo) {
                        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
                        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
                        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
                        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
                        const bool g_lo = (mx_lo - m_lo) * c2 > RESCALE_LOG2, g_hi = (mx_hi - m_hi) * c2 > RESCALE_LOG2;   // true from -inf
                        const bool f_lo = g_lo && m_lo != -INFINITY, f_hi = g_hi && m_hi != -INFINITY;   // O holds something to rescale
                        if (__any_sync(0xffffffffu, f_lo || f_hi)) {
                            // O must be at rest: wait for P(n-1) V, which by the issue order of the products also
                            // tells that every earlier one is done
                            if (!(ok = wait_warp(bPVt + 8 * ((n - 1) & 1), ((n - 1) >> 1) & 1))) break;
                            tc_fence_after();
                            const float a_lo = f_lo ? ex2((m_lo - mx_lo) * c2) : 1.f, a_hi = f_hi ? ex2((m_hi - mx_hi) * c2) : 1.f;
                            l0 *= a_lo; l1 *= a_lo; l2 *= a_hi; l3 *= a_hi;
                            uint32_t o[16];
#pragma unroll
                            for (int ch = 0; ch < D / 32; ++ch) {
                                tmem_ld16x256_x4(tO + ch * 32, o);
                                tc_wait_ld();
#pragma unroll
                                for (int e = 0; e < 16; ++e)
                                    o[e] = __float_as_uint(__uint_as_float(o[e]) * ((e & 2) ? a_hi : a_lo));
                                tmem_st16x256_x4(tO + ch * 32, o);
                            }
                        }
                        if (g_lo) m_lo = mx_lo;
                        if (g_hi) m_hi = mx_hi;
                    }
                } while (redo);
                if (!ok) break;
                l0 += b0; l1 += b1; l2 += b2; l3 += b3;
            } else {
#pragma unroll
                for (int e = 0; e < 16; ++e) pk[e] = 0u;
            }
            tmem_st16x128_x8(tS, pk);
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bPFt + 8 * buf);
            ++n;
        }
        // epilogue: O / l -> bf16 -> the tile's (now unused) Q buffer in the 128-byte swizzled layout
        // of the tensor map -> TMA stores, one per (query block, 64-channel half); rows past the
        // end of the sequence are clipped by the store
        if (ok && n > 0) ok = wait_warp(bOD + 8 * t, 0);
        if (ok) {
            tc_fence_after();
            float s_lo = l0 + l1, s_hi = l2 + l3;      // the quad's four partial sums make the row sum
            s_lo += __shfl_xor_sync(0xffffffffu, s_lo, 1);
            s_hi += __shfl_xor_sync(0xffffffffu, s_hi, 1);
            s_lo += __shfl_xor_sync(0xffffffffu, s_lo, 2);
            s_hi += __shfl_xor_sync(0xffffffffu, s_hi, 2);
            const float inv_lo = s_lo > 0.f ? 1.f / s_lo : 0.f, inv_hi = s_hi > 0.f ? 1.f / s_hi : 0.f;
            uint8_t* so_lo = smem + t * C::QTILE_BYTES + row_lo * 128;
            uint8_t* so_hi = so_lo + 8 * 128;
            const int sw_lo = row_lo & 7, sw_hi = (row_lo + 8) & 7;
            uint32_t o[16];
#pragma unroll
            for (int ch = 0; ch < D / 32; ++ch) {
                if (n > 0) {
                    tmem_ld16x256_x4(tO + ch * 32, o);
                    tc_wait_ld();
                } else {
#pragma unroll
                    for (int e = 0; e < 16; ++e) o[e] = 0u;
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    // channels 32 ch + 8 k + 2 cg, + 1: 16-byte chunk (4 (ch & 1) + k) of the 128-byte half row
                    const int chunk = (ch & 1) * 4 + k;
                    const uint32_t w_lo = pack_bf16(__uint_as_float(o[4 * k]) * inv_lo, __uint_as_float(o[4 * k + 1]) * inv_lo);
                    const uint32_t w_hi = pack_bf16(__uint_as_float(o[4 * k + 2]) * inv_hi, __uint_as_float(o[4 * k + 3]) * inv_hi);
                    *reinterpret_cast<uint32_t*>(so_lo + (ch >> 1) * QHALF_BYTES + ((chunk ^ sw_lo) << 4) + 4 * cg) = w_lo;
                    *reinterpret_cast<uint32_t*>(so_hi + (ch >> 1) * QHALF_BYTES + ((chunk ^ sw_hi) << 4) + 4 * cg) = w_hi;
                }
            }
            fence_proxy_async_smem();
        }
        // the four warps of a query block meet, then one lane stores the block
        const int qb_id = a;
        named_barrier_sync(1 + qb_id, 128);
        if (ok && (wl & 1) == 0 && hf == 0 && lane == 0 && qblk(qb_id) * 64 < N) {
#pragma unroll
            for (int dh = 0; dh < DH; ++dh)
                tma_store_4d(&tmo, sQ + t * C::QTILE_BYTES + dh * QHALF_BYTES + (wl >> 1) * BLK_BYTES, dh * 64,
                             qblk(qb_id) * 64, g.h0 + h, b);
            bulk_commit_group();
            bulk_wait_read_all();
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp >= MMA_WARP0) {
        if (ctl->abort_flag) {
            // make sure no UMMA of this warp is still in flight before the TMEM columns are released
            const uint32_t bT = smem_u32(&ctl->drain[warp - MMA_WARP0]);
            if (elect_one()) {
                tc_commit(bT);
                mbar_wait(bT, 0, 1u << 20);
            }
            __syncwarp();
        }
    }
    __syncthreads();
    if (warp == MMA_WARP0) {
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
    e = cudaFuncSetAttribute(attn_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)attn_smem_bytes<128>());
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)attn_smem_bytes<64>());
    if (e != cudaSuccess) return e;
    g_attr_set = true;
    return cudaSuccess;
}

cudaError_t launch_attention(const CUtensorMap& tmq, const CUtensorMap& tmk, const CUtensorMap& tmv,
                             const CUtensorMap& tmo,
                             const TensorGeom& g, const ImgList& imgs, const int32_t* kept_idx,
                             const int32_t* kept_cnt, const uint64_t* bitmask, float softmax_scale, int* status,
                             cudaStream_t s, const DevPlan* plan, int n_cap, int inject_stop_group, int pdl) {
    if (!g_attr_set) {
        cudaError_t e = attention_static_init();
        if (e != cudaSuccess) return e;
    }
    AttnParams prm;
    prm.g = g;
    prm.imgs = imgs;
    prm.kept_idx = kept_idx;
    prm.kept_cnt = kept_cnt;
    prm.bitmask32 = reinterpret_cast<const uint32_t*>(bitmask);
    prm.words32 = 2 * ((g.nb + 63) / 64);
    prm.status = status;
    prm.scale_log2 = softmax_scale * 1.4426950408889634f;
    int n_dense = 0;
    while (n_dense < imgs.n && (imgs.slot[n_dense] < 0 || kept_idx == nullptr)) ++n_dense;
    prm.n_dense = n_dense;
    prm.plan = plan;
    prm.stop_group = inject_stop_group;
    dim3 grid(((g.nb + 3) / 4) * g.H * (plan ? n_cap : imgs.n), 1, 1);
    if (inject_stop_group >= 0) {
        if (g.D == 128)
            attn_kernel<128, true><<<grid, NTHREADS, attn_smem_bytes<128>(), s>>>(tmq, tmk, tmv, tmo, prm);
        else
            attn_kernel<64, true><<<grid, NTHREADS, attn_smem_bytes<64>(), s>>>(tmq, tmk, tmv, tmo, prm);
    } else if (g.D == 128) {
        return launch_kernel(attn_kernel<128>, grid, dim3(NTHREADS), attn_smem_bytes<128>(), s, pdl != 0, tmq, tmk, tmv, tmo, prm);
    } else {
        return launch_kernel(attn_kernel<64>, grid, dim3(NTHREADS), attn_smem_bytes<64>(), s, pdl != 0, tmq, tmk, tmv, tmo, prm);
    }
    return cudaGetLastError();
}
