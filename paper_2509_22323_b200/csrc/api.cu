// Host side of the C ABI declared in rapid3.h: argument checks, workspace, tensor-map
// construction (cuTensorMapEncodeTiled through the runtime's driver entry point), the gate /
// compaction of rapid3_gated_step, and the kernel launches.
#include <math.h>
#include <string.h>

#include <new>
#include <vector>

#include "common.cuh"

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct MapSlot {
    const void* ptr = nullptr;
    CUtensorMap map;
};

struct ProfRec {
    cudaEvent_t a, b;
    int kind;
};

}  // namespace

struct rapid3_ctx {
    rapid3_shape shape;
    TensorGeom g;
    int words;                    // uint64 words per bitmask row
    // workspace (device)
    double* pooled = nullptr;     // [2][B_max][H][nb][D]
    float* scores = nullptr;      // [B_max][H][nb][nb]
    uint64_t* bitmask = nullptr;  // [B_max][H][nb][words]
    int32_t* kept_idx = nullptr;  // [B_max][H][nb][nb]
    int32_t* kept_cnt = nullptr;  // [B_max][H][nb]
    int32_t* row_keep = nullptr;  // [B_max][H][nb]: per-row counts of the cumulative-mass selection
    int* status = nullptr;
    DevPlan* plan = nullptr;      // device-resident plan of rapid3_gated_step_device
    // host-tensor staging of rapid3_gated_step_host (created on first use)
    void* stage[4] = {nullptr, nullptr, nullptr, nullptr};
    cudaStream_t up_s = nullptr, down_s = nullptr;            // copy streams of the host entry
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    std::vector<cudaEvent_t> ev_up, ev_done;                  // per image: inputs landed / output computed
    EncodeTiledFn encode = nullptr;
    MapSlot maps[8];              // small cache keyed by base pointer (round-robin replacement)
    int map_rr = 0;
    int64_t launches = 0;
    // optional per-kernel timing (rapid3_profile): event pairs around each launch
    int prof_mask = 0;            // bit k: launches of kernel kind k are bracketed by an event pair
    std::vector<ProfRec> prof;
    size_t prof_used = 0;
};

namespace {

enum { PROF_POOL = 0, PROF_SCORES, PROF_SELECT, PROF_ATTN };
#ifndef RAPID3_HOST_CHUNKS
#define RAPID3_HOST_CHUNKS 4
#endif
constexpr int HOST_CHUNKS = RAPID3_HOST_CHUNKS;     // head groups per image in the host-tensor entry's pipeline

// Records an event pair around one launch when profiling is on.
struct ProfScope {
    rapid3_ctx* c;
    cudaStream_t st;
    ProfRec* rec = nullptr;
    ProfScope(rapid3_ctx* ctx, int kind, cudaStream_t s) : c(ctx), st(s) {
        if (!((c->prof_mask >> kind) & 1)) return;
        if (c->prof_used == c->prof.size()) {
            if (c->prof.size() >= 16384) return;
            ProfRec r;
            if (cudaEventCreate(&r.a) != cudaSuccess) return;
            if (cudaEventCreate(&r.b) != cudaSuccess) { cudaEventDestroy(r.a); return; }
            c->prof.push_back(r);
        }
        rec = &c->prof[c->prof_used++];
        rec->kind = kind;
        cudaEventRecord(rec->a, st);
    }
    ~ProfScope() {
        if (rec) cudaEventRecord(rec->b, st);
    }
};

int keep_count(double ratio, int n_free) {
    double x = ceil(ratio * (double)n_free - 1e-6);
    if (x < 0) x = 0;
    if (x > n_free) x = n_free;
    return (int)x;
}

int check_shape(const rapid3_shape* s) {
    if (!s) return RAPID3_ERR_INVALID_ARG;
    if (s->block != 64) return RAPID3_ERR_UNSUPPORTED;
    if (s->D != 64 && s->D != 128) return RAPID3_ERR_UNSUPPORTED;
    if (s->B_max < 1 || s->B_max > RAPID3_MAX_IMG || s->H < 1 || s->H > 65535) return RAPID3_ERR_INVALID_ARG;
    if ((long long)s->B_max * s->H > 65535) return RAPID3_ERR_UNSUPPORTED;     // (image, head) pairs index a grid dimension
    if (s->n_text < 0 || s->n_image < 0) return RAPID3_ERR_INVALID_ARG;
    long long N = (long long)s->n_text + s->n_image;
    if (N < 1) return RAPID3_ERR_INVALID_ARG;
    if (N > 64ll * RAPID3_MAX_NB) return RAPID3_ERR_UNSUPPORTED;
    if (s->stride_n < s->D || s->stride_h < 1 || s->stride_b < 1) return RAPID3_ERR_INVALID_ARG;
    if ((s->stride_n % 8) || (s->stride_h % 8) || (s->stride_b % 8)) return RAPID3_ERR_INVALID_ARG;
    return RAPID3_OK;
}

int build_list(const rapid3_ctx* c, const int32_t* img_idx_host, int n_img, ImgList* l) {
    if (n_img < 1 || n_img > c->shape.B_max) return RAPID3_ERR_INVALID_ARG;
    l->n = n_img;
    for (int p = 0; p < n_img; ++p) {
        int b = img_idx_host ? img_idx_host[p] : p;
        if (b < 0 || b >= c->shape.B_max) return RAPID3_ERR_INVALID_ARG;
        l->batch[p] = b;
        l->slot[p] = p;
        l->k_free[p] = 0;
    }
    return RAPID3_OK;
}

// Tensor map over a bf16 [B, H, N, D] tensor: box = 64 channels x 64 tokens, 128-byte swizzle,
// out-of-range tokens read as zero.  The map is copied out by value at once: a later call may
// recycle the cache slot it came from.
int get_map(rapid3_ctx* c, const void* base, CUtensorMap* out) {
    for (auto& m : c->maps)
        if (m.ptr == base) { *out = m.map; return RAPID3_OK; }
    if (reinterpret_cast<uintptr_t>(base) % 16) return RAPID3_ERR_INVALID_ARG;
    constexpr int n_slots = (int)(sizeof(c->maps) / sizeof(c->maps[0]));
    MapSlot& m = c->maps[c->map_rr];
    c->map_rr = (c->map_rr + 1) % n_slots;
    const rapid3_shape& s = c->shape;
    cuuint64_t dims[4] = {(cuuint64_t)s.D, (cuuint64_t)c->g.N, (cuuint64_t)s.H, (cuuint64_t)s.B_max};
    cuuint64_t strides[3] = {(cuuint64_t)s.stride_n * 2, (cuuint64_t)s.stride_h * 2, (cuuint64_t)s.stride_b * 2};
    cuuint32_t box[4] = {64, 64, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    m.ptr = nullptr;
    CUresult r = c->encode(&m.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box,
                           estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return RAPID3_ERR_CUDA;
    m.ptr = base;
    *out = m.map;
    return RAPID3_OK;
}

// `g` is the context's geometry or a copy of it narrowed to a range of heads.
int attn_launch(rapid3_ctx* c, const TensorGeom& g, const void* q, const void* k, const void* v, void* out,
                const ImgList& l, const int32_t* kept_idx, const int32_t* kept_cnt, const uint64_t* bitmask, float scale,
                cudaStream_t st, const DevPlan* plan = nullptr, int n_cap = 0, bool after_select = false) {
    CUtensorMap tq, tk, tv, to;
    int r;
    if ((r = get_map(c, q, &tq)) || (r = get_map(c, k, &tk)) || (r = get_map(c, v, &tv)) || (r = get_map(c, out, &to)))
        return r;
    {
        ProfScope ps(c, PROF_ATTN, st);
        if (launch_attention(tq, tk, tv, to, g, l, kept_idx, kept_cnt, bitmask, scale, c->status, st, plan, n_cap, -1,
                             after_select) != cudaSuccess)
            return RAPID3_ERR_CUDA;
    }
    c->launches += 1;
    return RAPID3_OK;
}

}  // namespace

extern "C" {

const char* rapid3_strerror(int code) {
    switch (code) {
        case RAPID3_OK: return "ok";
        case RAPID3_ERR_INVALID_ARG: return "invalid argument";
        case RAPID3_ERR_UNSUPPORTED: return "unsupported shape";
        case RAPID3_ERR_WORKSPACE: return "workspace allocation failed or size limit exceeded";
        case RAPID3_ERR_CUDA: return "CUDA call failed";
        case RAPID3_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case RAPID3_ERR_BAD_LIST: return "kept-list entry out of range";
        default: return "unknown status";
    }
}

int rapid3_num_blocks(const rapid3_shape* s) {
    if (check_shape(s) != RAPID3_OK) return check_shape(s);
    return (int)(((long long)s->n_text + s->n_image + 63) / 64);
}

int rapid3_mask_words(const rapid3_shape* s) {
    int nb = rapid3_num_blocks(s);
    return nb < 0 ? nb : (nb + 63) / 64;
}

int rapid3_create(rapid3_ctx** out, const rapid3_shape* shape) {
    if (!out) return RAPID3_ERR_INVALID_ARG;
    *out = nullptr;
    int r = check_shape(shape);
    if (r != RAPID3_OK) return r;
    rapid3_ctx* c = new (std::nothrow) rapid3_ctx();
    if (!c) return RAPID3_ERR_WORKSPACE;
    c->shape = *shape;
    TensorGeom& g = c->g;
    g.H = shape->H;
    g.D = shape->D;
    g.N = shape->n_text + shape->n_image;
    g.nb = (g.N + 63) / 64;
    g.n_text_blocks = (shape->n_text + 63) / 64;
    // a 128 x 128 token grid after a block-aligned text prefix: one grid row = two blocks
    // and when the text prefix is a whole number of quads, a quad is one column of four grid rows
    g.h0 = 0;
    g.pair_stride = 1;
    if (shape->n_image == 128 * 128 && shape->n_text % 64 == 0) g.pair_stride = (g.n_text_blocks % 4 == 0) ? 3 : 2;
    g.stride_b = shape->stride_b;
    g.stride_h = shape->stride_h;
    g.stride_n = shape->stride_n;
    c->words = (g.nb + 63) / 64;

    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess) {
        delete c;
        return RAPID3_ERR_CUDA;
    }
    c->encode = reinterpret_cast<EncodeTiledFn>(fn);

    const size_t B = shape->B_max, H = g.H, nb = g.nb;
    bool ok = cudaMalloc(&c->pooled, 2 * B * H * nb * g.D * sizeof(double)) == cudaSuccess &&
              cudaMalloc(&c->scores, B * H * nb * nb * sizeof(float)) == cudaSuccess &&
              cudaMalloc(&c->bitmask, B * H * nb * c->words * sizeof(uint64_t)) == cudaSuccess &&
              cudaMalloc(&c->kept_idx, B * H * nb * nb * sizeof(int32_t)) == cudaSuccess &&
              cudaMalloc(&c->kept_cnt, B * H * nb * sizeof(int32_t)) == cudaSuccess &&
              cudaMalloc(&c->row_keep, B * H * nb * sizeof(int32_t)) == cudaSuccess &&
              cudaMalloc(&c->status, sizeof(int)) == cudaSuccess &&
              cudaMemset(c->status, 0, sizeof(int)) == cudaSuccess &&
              cudaMalloc(&c->plan, sizeof(DevPlan)) == cudaSuccess &&
              cudaMemset(c->plan, 0, sizeof(DevPlan)) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        rapid3_destroy(c);
        return RAPID3_ERR_WORKSPACE;
    }
    if (attention_static_init() != cudaSuccess) {
        cudaGetLastError();
        rapid3_destroy(c);
        return RAPID3_ERR_CUDA;
    }
    *out = c;
    return RAPID3_OK;
}

int rapid3_destroy(rapid3_ctx* c) {
    if (!c) return RAPID3_ERR_INVALID_ARG;
    cudaFree(c->pooled);
    cudaFree(c->scores);
    cudaFree(c->bitmask);
    cudaFree(c->kept_idx);
    cudaFree(c->kept_cnt);
    cudaFree(c->row_keep);
    cudaFree(c->status);
    cudaFree(c->plan);
    for (void* s : c->stage) cudaFree(s);
    if (c->up_s) cudaStreamDestroy(c->up_s);
    if (c->down_s) cudaStreamDestroy(c->down_s);
    if (c->ev_fork) cudaEventDestroy(c->ev_fork);
    if (c->ev_join) cudaEventDestroy(c->ev_join);
    for (cudaEvent_t e : c->ev_up) cudaEventDestroy(e);
    for (cudaEvent_t e : c->ev_done) cudaEventDestroy(e);
    for (auto& r : c->prof) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    delete c;
    return RAPID3_OK;
}

int rapid3_block_scores(rapid3_ctx* c, const void* q, const void* k, const int32_t* img_idx_host, int n_img,
                        float* scores, void* stream) {
    if (!c || !q || !k || !scores) return RAPID3_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(q) % 16) || (reinterpret_cast<uintptr_t>(k) % 16)) return RAPID3_ERR_INVALID_ARG;
    ImgList l;
    int r = build_list(c, img_idx_host, n_img, &l);
    if (r != RAPID3_OK) return r;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    {
        ProfScope ps(c, PROF_POOL, st);
        if (launch_block_pool(q, k, c->g, l, c->pooled, st) != cudaSuccess) return RAPID3_ERR_CUDA;
    }
    {
        ProfScope ps(c, PROF_SCORES, st);
        if (launch_block_scores(c->pooled, c->g, n_img, scores, st, nullptr, true) != cudaSuccess) return RAPID3_ERR_CUDA;
    }
    c->launches += 2;
    return RAPID3_OK;
}

int rapid3_select_mask(rapid3_ctx* c, const float* scores, const float* keep_ratio_host, int n_img,
                       uint64_t* bitmask, int32_t* kept_idx, int32_t* kept_cnt, void* stream) {
    if (!c || !scores || !keep_ratio_host || !bitmask || !kept_idx || !kept_cnt) return RAPID3_ERR_INVALID_ARG;
    ImgList l;
    int r = build_list(c, nullptr, n_img, &l);
    if (r != RAPID3_OK) return r;
    const int n_free_img = c->g.nb - c->g.n_text_blocks - 1;   // free candidates of an image query row
    for (int p = 0; p < n_img; ++p) {
        const float ratio = keep_ratio_host[p];
        if (!(ratio > 0.f) || !(ratio <= 1.f)) return RAPID3_ERR_INVALID_ARG;
        l.k_free[p] = keep_count((double)ratio, n_free_img > 0 ? n_free_img : 0);
    }
    {
        ProfScope ps(c, PROF_SELECT, static_cast<cudaStream_t>(stream));
        if (launch_select_mask(scores, c->g, l, bitmask, kept_idx, kept_cnt, static_cast<cudaStream_t>(stream)) !=
            cudaSuccess)
            return RAPID3_ERR_CUDA;
    }
    c->launches += 1;
    return RAPID3_OK;
}

int rapid3_select_mask_mass(rapid3_ctx* c, const float* scores, const float* mass_share_host, float mass_scale,
                            int n_img, int32_t* row_keep, uint64_t* bitmask, int32_t* kept_idx, int32_t* kept_cnt,
                            void* stream) {
    if (!c || !scores || !mass_share_host || !row_keep || !bitmask || !kept_idx || !kept_cnt) return RAPID3_ERR_INVALID_ARG;
    if (!(mass_scale >= 0.f) || !isfinite(mass_scale)) return RAPID3_ERR_INVALID_ARG;
    ImgList l;
    int r = build_list(c, nullptr, n_img, &l);
    if (r != RAPID3_OK) return r;
    MassShare share;
    for (int p = 0; p < n_img; ++p) {
        const float tau = mass_share_host[p];
        if (!(tau > 0.f) || !(tau <= 1.f)) return RAPID3_ERR_INVALID_ARG;
        share.tau[p] = tau;
        l.k_free[p] = 0;
    }
    {
        ProfScope ps(c, PROF_SELECT, static_cast<cudaStream_t>(stream));
        if (launch_select_mask_mass(scores, c->g, l, share, mass_scale, row_keep, bitmask, kept_idx, kept_cnt,
                                    static_cast<cudaStream_t>(stream)) != cudaSuccess)
            return RAPID3_ERR_CUDA;
    }
    c->launches += 2;
    return RAPID3_OK;
}

int rapid3_sparse_joint_attn(rapid3_ctx* c, const void* q, const void* k, const void* v, void* out,
                             const int32_t* img_idx_host, int n_img, const int32_t* kept_idx,
                             const int32_t* kept_cnt, float softmax_scale, void* stream) {
    if (!c || !q || !k || !v || !out) return RAPID3_ERR_INVALID_ARG;
    if ((kept_idx == nullptr) != (kept_cnt == nullptr)) return RAPID3_ERR_INVALID_ARG;
    if (!(softmax_scale > 0.f) || !isfinite(softmax_scale)) return RAPID3_ERR_INVALID_ARG;
    ImgList l;
    int r = build_list(c, img_idx_host, n_img, &l);
    if (r != RAPID3_OK) return r;
    if (!kept_idx)
        for (int p = 0; p < n_img; ++p) l.slot[p] = -1;
    return attn_launch(c, c->g, q, k, v, out, l, kept_idx, kept_cnt, nullptr, softmax_scale,
                       static_cast<cudaStream_t>(stream));
}

// One gated step.  heads_per_ratio == 1: keep_ratio_host is [B].  heads_per_ratio == H: it is
// [B][H], one ratio per (image, head); an image is dense only when all its heads keep everything.
// With `prep` set, Q and K are first produced from prep->q_raw / k_raw into q / k by the fused
// producer, which also writes the block means: the pooling kernel is then not launched.
// With `heads` set, only heads [heads->first, heads->first + heads->count) of the tensors are processed
// (heads are independent; the workspace then holds that many heads, counted from 0).
struct HeadRange {
    int first, count;
};
static int gated_step_impl(rapid3_ctx* c, const void* q, const void* k, const void* v, void* out,
                           const int32_t* action_host, const float* keep_ratio_host, int heads_per_ratio, int B,
                           float softmax_scale, void* stream, const PrepArgs* prep = nullptr,
                           const float* mass_scale = nullptr, const HeadRange* heads = nullptr) {
    if (!c || !q || !k || !v || !out || !action_host || !keep_ratio_host) return RAPID3_ERR_INVALID_ARG;
    if (B < 1 || B > c->shape.B_max) return RAPID3_ERR_INVALID_ARG;
    if (!(softmax_scale > 0.f) || !isfinite(softmax_scale)) return RAPID3_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    TensorGeom g = c->g;
    if (heads) {
        if (heads->first < 0 || heads->count < 1 || heads->first + heads->count > c->g.H) return RAPID3_ERR_INVALID_ARG;
        g.h0 = heads->first;
        g.H = heads->count;
    }
    const int n_free_img = g.nb - g.n_text_blocks - 1;
    // gate + compaction: sparse images (ascending batch order) get workspace slots 0..ns-1;
    // the attention list puts dense images first (longest work first), then sparse by ratio
    ImgList sparse, all;
    sparse.n = 0;
    all.n = 0;
    float ratio_of[RAPID3_MAX_IMG];
    // with mass_scale set, keep_ratio_host holds mass shares and the selection is the cumulative-mass rule
    const bool per_head = heads_per_ratio > 1;
    const int H = g.H;
    HeadKeep hk;
    MassShare share;
    if (per_head) memset(&hk, 0, sizeof hk);
    for (int b = 0; b < B; ++b) {
        const int a = action_host[b];
        if (a != RAPID3_ACT_SKIP && a != RAPID3_ACT_REUSE && a != RAPID3_ACT_ATTEND) return RAPID3_ERR_INVALID_ARG;
        if (a != RAPID3_ACT_ATTEND) continue;
        float ratio = keep_ratio_host[(size_t)b * heads_per_ratio];
        if (per_head) {                                   // order images by their mean ratio
            double sum = 0.0;
            bool all_one = true;
            for (int h = 0; h < H; ++h) {
                const float rh = keep_ratio_host[(size_t)b * H + h];
                if (!(rh > 0.f) || !(rh <= 1.f)) return RAPID3_ERR_INVALID_ARG;
                sum += rh;
                all_one = all_one && rh == 1.f;
            }
            ratio = all_one ? 1.f : fminf((float)(sum / H), 0.99999994f);
        }
        if (!(ratio > 0.f) || !(ratio <= 1.f)) return RAPID3_ERR_INVALID_ARG;
        int slot = -1;
        if (ratio < 1.f) {
            slot = sparse.n++;
            sparse.batch[slot] = b;
            sparse.slot[slot] = slot;
            sparse.k_free[slot] = keep_count((double)ratio, n_free_img > 0 ? n_free_img : 0);
            share.tau[slot] = ratio;
            if (per_head) {
                if ((slot + 1) * H > RAPID3_MAX_HEAD_ROWS) return RAPID3_ERR_UNSUPPORTED;
                for (int h = 0; h < H; ++h)
                    hk.k[slot * H + h] =
                        keep_count((double)keep_ratio_host[(size_t)b * H + h], n_free_img > 0 ? n_free_img : 0);
            }
        }
        int pos = all.n++;
        while (pos > 0 && ratio_of[pos - 1] < ratio) {   // insertion sort, descending ratio, stable
            all.batch[pos] = all.batch[pos - 1];
            all.slot[pos] = all.slot[pos - 1];
            ratio_of[pos] = ratio_of[pos - 1];
            --pos;
        }
        all.batch[pos] = b;
        all.slot[pos] = slot;
        all.k_free[pos] = 0;
        ratio_of[pos] = ratio;
    }
    if (all.n == 0) return RAPID3_OK;                     // every image gated: nothing is launched
    if (prep) {
        ProfScope ps(c, PROF_POOL, st);
        if (launch_prepare(*prep, g, all, sparse.n, c->pooled, st) != cudaSuccess) return RAPID3_ERR_CUDA;
        c->launches += 1;
    }
    if (sparse.n > 0) {
        if ((reinterpret_cast<uintptr_t>(q) % 16) || (reinterpret_cast<uintptr_t>(k) % 16)) return RAPID3_ERR_INVALID_ARG;
        if (!prep) {
            ProfScope ps(c, PROF_POOL, st);
            if (launch_block_pool(q, k, g, sparse, c->pooled, st) != cudaSuccess) return RAPID3_ERR_CUDA;
            c->launches += 1;
        }
        {
            ProfScope ps(c, PROF_SCORES, st);
            if (launch_block_scores(c->pooled, g, sparse.n, c->scores, st, nullptr, true) != cudaSuccess) return RAPID3_ERR_CUDA;
        }
        {
            ProfScope ps(c, PROF_SELECT, st);
            const cudaError_t e =
                mass_scale ? launch_select_mask_mass(c->scores, g, sparse, share, *mass_scale, c->row_keep, c->bitmask,
                                                     c->kept_idx, c->kept_cnt, st)
                : per_head ? launch_select_mask_heads(c->scores, g, sparse, hk, c->bitmask, c->kept_idx, c->kept_cnt, st, true)
                           : launch_select_mask(c->scores, g, sparse, c->bitmask, c->kept_idx, c->kept_cnt, st, nullptr, 0, true);
            if (e != cudaSuccess) return RAPID3_ERR_CUDA;
        }
        c->launches += mass_scale ? 3 : 2;
    }
    return attn_launch(c, g, q, k, v, out, all, sparse.n ? c->kept_idx : nullptr, sparse.n ? c->kept_cnt : nullptr,
                       sparse.n ? c->bitmask : nullptr, softmax_scale, st, nullptr, 0, sparse.n > 0 && !mass_scale);
}

int rapid3_gated_step(rapid3_ctx* c, const void* q, const void* k, const void* v, void* out,
                      const int32_t* action_host, const float* keep_ratio_host, int B, float softmax_scale,
                      void* stream) {
    return gated_step_impl(c, q, k, v, out, action_host, keep_ratio_host, 1, B, softmax_scale, stream);
}

int rapid3_gated_step_mass(rapid3_ctx* c, const void* q, const void* k, const void* v, void* out,
                           const int32_t* action_host, const float* mass_share_host, float mass_scale, int B,
                           float softmax_scale, void* stream) {
    if (!(mass_scale >= 0.f) || !isfinite(mass_scale)) return RAPID3_ERR_INVALID_ARG;
    return gated_step_impl(c, q, k, v, out, action_host, mass_share_host, 1, B, softmax_scale, stream, nullptr,
                           &mass_scale);
}

int rapid3_gated_step_fused(rapid3_ctx* c, const void* q_raw, const void* k_raw, const void* v, const float* q_gain,
                            const float* k_gain, const float* rot, float eps, void* q, void* k, void* out,
                            const int32_t* action_host, const float* keep_ratio_host, int B, float softmax_scale,
                            void* stream) {
    if (!c || !q_raw || !k_raw || !q_gain || !k_gain || !q || !k) return RAPID3_ERR_INVALID_ARG;
    if (!(eps >= 0.f) || !isfinite(eps)) return RAPID3_ERR_INVALID_ARG;
    const uintptr_t al = reinterpret_cast<uintptr_t>(q_raw) | reinterpret_cast<uintptr_t>(k_raw) |
                         reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k) |
                         reinterpret_cast<uintptr_t>(q_gain) | reinterpret_cast<uintptr_t>(k_gain) |
                         reinterpret_cast<uintptr_t>(rot);
    if (al % 16) return RAPID3_ERR_INVALID_ARG;
    PrepArgs prep{q_raw, k_raw, q, k, q_gain, k_gain, rot, eps};
    return gated_step_impl(c, q, k, v, out, action_host, keep_ratio_host, 1, B, softmax_scale, stream, &prep);
}

int rapid3_gated_step_heads(rapid3_ctx* c, const void* q, const void* k, const void* v, void* out,
                            const int32_t* action_host, const float* keep_ratio_host, int B, float softmax_scale,
                            void* stream) {
    if (!c) return RAPID3_ERR_INVALID_ARG;
    if (c->g.H == 1)
        return gated_step_impl(c, q, k, v, out, action_host, keep_ratio_host, 1, B, softmax_scale, stream);
    return gated_step_impl(c, q, k, v, out, action_host, keep_ratio_host, c->g.H, B, softmax_scale, stream);
}

int rapid3_gated_step_device(rapid3_ctx* c, const void* q, const void* k, const void* v, void* out,
                             const int32_t* action_dev, const float* keep_ratio_dev, int B, float softmax_scale,
                             void* stream) {
    if (!c || !q || !k || !v || !out || !action_dev || !keep_ratio_dev) return RAPID3_ERR_INVALID_ARG;
    if (B < 1 || B > c->shape.B_max) return RAPID3_ERR_INVALID_ARG;
    if (!(softmax_scale > 0.f) || !isfinite(softmax_scale)) return RAPID3_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(q) % 16) || (reinterpret_cast<uintptr_t>(k) % 16)) return RAPID3_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The host never sees the actions: a one-thread kernel does the gate and compaction into the
    // context's device-resident plan, and every following kernel is launched with a grid that covers
    // all B images and takes its image list from the plan; the surplus CTAs return at once.
    if (launch_plan(action_dev, keep_ratio_dev, B, c->g, c->plan, c->status, st) != cudaSuccess) return RAPID3_ERR_CUDA;
    ImgList none;
    none.n = 0;
    {
        ProfScope ps(c, PROF_POOL, st);
        if (launch_block_pool(q, k, c->g, none, c->pooled, st, c->plan, B) != cudaSuccess) return RAPID3_ERR_CUDA;
    }
    {
        ProfScope ps(c, PROF_SCORES, st);
        if (launch_block_scores(c->pooled, c->g, B, c->scores, st, c->plan) != cudaSuccess) return RAPID3_ERR_CUDA;
    }
    {
        ProfScope ps(c, PROF_SELECT, st);
        if (launch_select_mask(c->scores, c->g, none, c->bitmask, c->kept_idx, c->kept_cnt, st, c->plan, B) != cudaSuccess)
            return RAPID3_ERR_CUDA;
    }
    c->launches += 4;
    return attn_launch(c, c->g, q, k, v, out, none, c->kept_idx, c->kept_cnt, c->bitmask, softmax_scale, st, c->plan, B);
}

int rapid3_gated_step_host(rapid3_ctx* c, const void* q_host, const void* k_host, const void* v_host, void* out_host,
                           const int32_t* action_host, const float* keep_ratio_host, int B, float softmax_scale,
                           void* stream, int64_t* bytes_h2d, int64_t* bytes_d2h) {
    if (!c || !q_host || !k_host || !v_host || !out_host || !action_host || !keep_ratio_host)
        return RAPID3_ERR_INVALID_ARG;
    if (B < 1 || B > c->shape.B_max) return RAPID3_ERR_INVALID_ARG;
    const rapid3_shape& s = c->shape;
    const long long N = c->g.N;
    // staging is contiguous [B, H, N, D]; the context's strides must describe exactly that
    if (s.stride_n != s.D || s.stride_h != N * s.D || s.stride_b != (long long)s.H * N * s.D)
        return RAPID3_ERR_UNSUPPORTED;
    const size_t img_bytes = (size_t)s.H * N * s.D * 2;
    for (int b = 0; b < B; ++b) {
        const int a = action_host[b];
        if (a != RAPID3_ACT_SKIP && a != RAPID3_ACT_REUSE && a != RAPID3_ACT_ATTEND) return RAPID3_ERR_INVALID_ARG;
        if (a == RAPID3_ACT_ATTEND && (!(keep_ratio_host[b] > 0.f) || !(keep_ratio_host[b] <= 1.f)))
            return RAPID3_ERR_INVALID_ARG;
    }
    if (!(softmax_scale > 0.f) || !isfinite(softmax_scale)) return RAPID3_ERR_INVALID_ARG;
    if (!c->stage[0]) {
        bool ok = true;
        for (int i = 0; i < 4 && ok; ++i) ok = cudaMalloc(&c->stage[i], img_bytes * s.B_max) == cudaSuccess;
        ok = ok && cudaStreamCreateWithFlags(&c->up_s, cudaStreamNonBlocking) == cudaSuccess &&
             cudaStreamCreateWithFlags(&c->down_s, cudaStreamNonBlocking) == cudaSuccess &&
             cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) == cudaSuccess;
        for (int b = 0; b < s.B_max * HOST_CHUNKS && ok; ++b) {
            cudaEvent_t e0 = nullptr, e1 = nullptr;
            ok = cudaEventCreateWithFlags(&e0, cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&e1, cudaEventDisableTiming) == cudaSuccess;
            if (e0) c->ev_up.push_back(e0);
            if (e1) c->ev_done.push_back(e1);
        }
        if (!ok) {
            cudaGetLastError();
            for (int j = 0; j < 4; ++j) { cudaFree(c->stage[j]); c->stage[j] = nullptr; }
            return RAPID3_ERR_WORKSPACE;
        }
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const void* src[3] = {q_host, k_host, v_host};
    int64_t up = 0, down = 0;
    // Image by image: inputs go up on one copy stream, the step of that image runs on `stream` as soon as
    // they have landed, its output goes down on a second copy stream -- so the uploads of the next images,
    // the compute and the downloads overlap (the link is full duplex).  The last image goes in
    // HOST_CHUNKS groups of heads (heads are independent), so that what is left after the last upload is
    // one small group's compute and download.  Everything is forked from and joined back into `stream`.
    if (cudaEventRecord(c->ev_fork, st) != cudaSuccess || cudaStreamWaitEvent(c->up_s, c->ev_fork, 0) != cudaSuccess ||
        cudaStreamWaitEvent(c->down_s, c->ev_fork, 0) != cudaSuccess)
        return RAPID3_ERR_CUDA;
    int32_t one[RAPID3_MAX_IMG];
    for (int b = 0; b < B; ++b) one[b] = RAPID3_ACT_SKIP;
    bool any = false;
    // only the last attending image is cut into head groups: every copy costs a few microseconds of
    // engine turnaround, and it is the last image's compute and download that nothing overlaps
    int last = -1;
    for (int b = 0; b < B; ++b)
        if (action_host[b] == RAPID3_ACT_ATTEND) last = b;
    const int H_all = s.H;
    const size_t head_bytes = (size_t)N * s.D * 2;
    for (int b = 0; b < B; ++b) {
        if (action_host[b] != RAPID3_ACT_ATTEND) continue;
        any = true;
        const int heads_per_chunk = (b == last) ? (H_all + HOST_CHUNKS - 1) / HOST_CHUNKS : H_all;
        for (int h0 = 0, ch = 0; h0 < H_all; h0 += heads_per_chunk, ++ch) {
            const int hn = (H_all - h0 < heads_per_chunk) ? H_all - h0 : heads_per_chunk;
            const size_t off = b * img_bytes + h0 * head_bytes, bytes = hn * head_bytes;
            cudaEvent_t e_up = c->ev_up[b * HOST_CHUNKS + ch], e_done = c->ev_done[b * HOST_CHUNKS + ch];
            for (int i = 0; i < 3; ++i) {
                if (cudaMemcpyAsync((char*)c->stage[i] + off, (const char*)src[i] + off, bytes, cudaMemcpyHostToDevice,
                                    c->up_s) != cudaSuccess)
                    return RAPID3_ERR_CUDA;
                up += (int64_t)bytes;
            }
            if (cudaEventRecord(e_up, c->up_s) != cudaSuccess || cudaStreamWaitEvent(st, e_up, 0) != cudaSuccess)
                return RAPID3_ERR_CUDA;
            // heads h0 .. h0 + hn of image b alone: every other image is given the skip action
            one[b] = RAPID3_ACT_ATTEND;
            const HeadRange hr{h0, hn};
            const int r = gated_step_impl(c, c->stage[0], c->stage[1], c->stage[2], c->stage[3], one, keep_ratio_host, 1,
                                          B, softmax_scale, stream, nullptr, nullptr, &hr);
            one[b] = RAPID3_ACT_SKIP;
            if (r != RAPID3_OK) return r;
            if (cudaEventRecord(e_done, st) != cudaSuccess || cudaStreamWaitEvent(c->down_s, e_done, 0) != cudaSuccess)
                return RAPID3_ERR_CUDA;
            if (cudaMemcpyAsync((char*)out_host + off, (const char*)c->stage[3] + off, bytes, cudaMemcpyDeviceToHost,
                                c->down_s) != cudaSuccess)
                return RAPID3_ERR_CUDA;
            down += (int64_t)bytes;
        }
    }
    if (any && (cudaEventRecord(c->ev_join, c->down_s) != cudaSuccess || cudaStreamWaitEvent(st, c->ev_join, 0) != cudaSuccess))
        return RAPID3_ERR_CUDA;
    if (bytes_h2d) *bytes_h2d = up;
    if (bytes_d2h) *bytes_d2h = down;
    return RAPID3_OK;
}

int rapid3_debug_inject_timeout(rapid3_ctx* c, const void* q, const void* k, const void* v, void* out, int stop_group,
                                float softmax_scale, void* stream) {
    if (!c || !q || !k || !v || !out) return RAPID3_ERR_INVALID_ARG;
    if (stop_group < 0 || stop_group > c->g.nb) return RAPID3_ERR_INVALID_ARG;
    if (!(softmax_scale > 0.f) || !isfinite(softmax_scale)) return RAPID3_ERR_INVALID_ARG;
    ImgList l;
    l.n = 1;
    l.batch[0] = 0;
    l.slot[0] = -1;                                       // dense: every CTA walks all nb key blocks
    l.k_free[0] = 0;
    CUtensorMap tq, tk, tv, to;
    int r;
    if ((r = get_map(c, q, &tq)) || (r = get_map(c, k, &tk)) || (r = get_map(c, v, &tv)) || (r = get_map(c, out, &to)))
        return r;
    if (launch_attention(tq, tk, tv, to, c->g, l, nullptr, nullptr, nullptr, softmax_scale, c->status,
                         static_cast<cudaStream_t>(stream), nullptr, 0, stop_group) != cudaSuccess)
        return RAPID3_ERR_CUDA;
    c->launches += 1;
    return RAPID3_OK;
}

int rapid3_workspace(rapid3_ctx* c, float** scores, uint64_t** bitmask, int32_t** kept_idx, int32_t** kept_cnt) {
    if (!c) return RAPID3_ERR_INVALID_ARG;
    if (scores) *scores = c->scores;
    if (bitmask) *bitmask = c->bitmask;
    if (kept_idx) *kept_idx = c->kept_idx;
    if (kept_cnt) *kept_cnt = c->kept_cnt;
    return RAPID3_OK;
}

int64_t rapid3_launch_count(rapid3_ctx* c) { return c ? c->launches : -1; }

int rapid3_profile(rapid3_ctx* c, int enable) {
    if (!c) return RAPID3_ERR_INVALID_ARG;
    if (enable < 0 || enable > 2) return RAPID3_ERR_INVALID_ARG;
    c->prof_mask = enable == 1 ? 0xF : (enable == 2 ? (1 << PROF_ATTN) : 0);
    return RAPID3_OK;
}

int rapid3_profile_read(rapid3_ctx* c, double* ms, int64_t* launches) {
    if (!c || !ms || !launches) return RAPID3_ERR_INVALID_ARG;
    for (int i = 0; i < 4; ++i) { ms[i] = 0.0; launches[i] = 0; }
    for (size_t i = 0; i < c->prof_used; ++i) {
        ProfRec& r = c->prof[i];
        float t = 0.f;
        if (cudaEventSynchronize(r.b) != cudaSuccess || cudaEventElapsedTime(&t, r.a, r.b) != cudaSuccess)
            return RAPID3_ERR_CUDA;
        ms[r.kind] += (double)t;
        launches[r.kind] += 1;
    }
    c->prof_used = 0;
    return RAPID3_OK;
}

int rapid3_last_status(rapid3_ctx* c, int* device_status) {
    if (!c || !device_status) return RAPID3_ERR_INVALID_ARG;
    int v = 0;
    if (cudaMemcpy(&v, c->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return RAPID3_ERR_CUDA;
    if (v != 0 && cudaMemset(c->status, 0, sizeof(int)) != cudaSuccess) return RAPID3_ERR_CUDA;
    *device_status = v;
    return RAPID3_OK;
}

}  // extern "C"

int rapid3_equivalent_steps(const int32_t* action_host, const float* c_cache_host, const float* c_sparse_host,
                            int n_steps, double* k_exact, int64_t* k_rounded) {
    if (n_steps < 0 || (n_steps > 0 && (!action_host || !c_cache_host || !c_sparse_host))) return RAPID3_ERR_INVALID_ARG;
    double sum = 0.0;
    for (int s = 0; s < n_steps; ++s) {
        const int a = action_host[s];
        if (a == RAPID3_ACT_SKIP) continue;
        const float c = a == RAPID3_ACT_REUSE ? c_cache_host[s] : c_sparse_host[s];
        if ((a != RAPID3_ACT_REUSE && a != RAPID3_ACT_ATTEND) || !(c >= 0.f) || !(c <= 1.f)) return RAPID3_ERR_INVALID_ARG;
        sum += 1.0 - (double)c;
    }
    if (k_exact) *k_exact = sum;
    if (k_rounded) *k_rounded = (int64_t)floor(sum + 0.5);
    return RAPID3_OK;
}
