/*
 * rapid3.h -- C ABI of the policy-gated block-sparse joint attention library (sm_100a).
 *
 * The hot path is the one the Sparse-Attention policy head of RAPID^3 accelerates
 * (paper Sec. 3.2 "Level-3: Sparse-Attention", Sec. 3.3 c): inside each MMDiT block of a
 * denoising step the joint (text + image token) self-attention is replaced by a sparse
 * attention whose sparsity level is chosen per image and per step by the policy; an image
 * whose Step-Skip (Sec. 3.2 "Level-1") or Cache-Reuse (Sec. 3.2 "Level-2", Sec. 3.3 b)
 * action fires runs no attention at all in that step.
 *
 * Sparsity rule (the paper leaves it to a third-party kernel; this library fixes it):
 *   - the joint sequence is text tokens first, then image tokens in raster order;
 *     it is cut into blocks of 64 tokens, nb = ceil(N / 64); the last block may be short;
 *   - block scores S[i][j] = mean(Q over block i) . mean(K over block j)   (no softmax scale);
 *   - a block that holds at least one text token is a "text block" (the first ceil(n_text/64));
 *   - query block i always keeps: every text block, and block i itself; a text query block
 *     keeps every block;
 *   - of its other ("free") blocks it keeps the k = min(n_free, ceil(ratio * n_free - 1e-6))
 *     with the highest score, ties broken towards the lower block index;
 *   - attention of a query token = softmax over exactly the valid tokens of the kept key
 *     blocks of its query block, times V.
 *
 * Conventions
 *   - Every `q`, `k`, `v`, `out`, `scores`, `bitmask`, `kept_idx`, `kept_cnt` pointer is a DEVICE
 *     pointer owned by the caller.  Every `*_host` pointer is a HOST pointer that is read
 *     before the call returns.
 *   - Q, K, V, O are bf16 tensors [B, H, N, D] addressed with the element strides of
 *     rapid3_shape (the D stride is 1).  Base pointers and row starts must be 16-byte aligned
 *     (strides multiples of 8 elements).
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*), never synchronise
 *     the host, and allocate nothing: all device workspace is created by rapid3_create.
 *     (Exception, documented below: rapid3_gated_step_host stages through buffers it creates
 *     on first use.)
 *   - Every function returns a status code; nothing throws, prints or aborts.  Problems that
 *     only the device can see (a bounded wait that ran out, a kept-list entry out of range)
 *     are recorded in a device status word, read with rapid3_last_status.
 *   - Non-finite inputs give undefined results.
 *   - A context is used by one host thread at a time and its calls are ordered on the stream(s)
 *     they are given: its workspace (block means, scores, masks, lists) is shared by all its
 *     calls, so two calls of one context on different streams must be ordered by the caller.
 *     Different contexts are independent (also on one device, on different streams) and a
 *     context belongs to the device that was current when it was created.
 */
#ifndef RAPID3_H_
#define RAPID3_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct rapid3_ctx rapid3_ctx; /* opaque: workspace, tensor-map cache, status word */

typedef struct rapid3_shape {
    int32_t B_max;    /* largest batch a call may pass (1..64)                        */
    int32_t H;        /* heads (B_max * H <= 65535, else RAPID3_ERR_UNSUPPORTED)      */
    int32_t D;        /* head dimension: 64 or 128                                    */
    int32_t n_text;   /* text tokens (>= 0), first in the joint sequence              */
    int32_t n_image;  /* image tokens (>= 0), after the text tokens; N = n_text+n_image, 1..65536 */
    int32_t block;    /* must be 64                                                   */
    int64_t stride_b; /* element strides of Q, K, V and O; all four tensors share them */
    int64_t stride_h;
    int64_t stride_n;
} rapid3_shape;

enum {
    RAPID3_OK = 0,
    RAPID3_ERR_INVALID_ARG = -1, /* null pointer, bad count, ratio outside (0, 1], ...   */
    RAPID3_ERR_UNSUPPORTED = -2, /* shape the kernels do not cover                       */
    RAPID3_ERR_WORKSPACE = -3,   /* device allocation failed / size limit exceeded       */
    RAPID3_ERR_CUDA = -4,        /* a CUDA runtime or driver call failed                 */
    RAPID3_ERR_TIMEOUT = -5,     /* device status: a bounded wait inside a kernel ran out */
    RAPID3_ERR_BAD_LIST = -6     /* device status: a kept-list entry was out of range    */
};

/* Per-image policy action of one step (Sec. 3.3: a^cache = 1 is a reuse, a skipped time
 * step never runs; only ATTEND launches attention work). */
enum { RAPID3_ACT_SKIP = 0, RAPID3_ACT_REUSE = 1, RAPID3_ACT_ATTEND = 2 };

/* Creates a context for one shape on the current device and allocates all device workspace
 * (pooled means, scores, masks and kept lists for B_max images).  *out is NULL on failure. */
int rapid3_create(rapid3_ctx** out, const rapid3_shape* shape);
/* Frees the workspace.  The caller makes sure no call using the context is still running. */
int rapid3_destroy(rapid3_ctx* ctx);
const char* rapid3_strerror(int code);

/* nb = ceil((n_text + n_image) / 64) and the number of uint64 words of one bitmask row. */
int rapid3_num_blocks(const rapid3_shape* shape);
int rapid3_mask_words(const rapid3_shape* shape);

/*
 * Stage (a), part 1: pooled block scores (sparsity rule above, steps "block scores").
 * For the n_img images whose batch indices are listed in img_idx_host (NULL means
 * 0..n_img-1), writes scores[p][h][i][j] (fp32, [n_img, H, nb, nb], compacted in list order).
 * Block means and the dot products are accumulated in fp64 and rounded once to fp32.
 * Reads Q and K once.
 */
int rapid3_block_scores(rapid3_ctx* ctx, const void* q, const void* k, const int32_t* img_idx_host,
                        int n_img, float* scores, void* stream);

/*
 * Stage (a), part 2: per (image, head, query block) forced + top-k block mask at each image's
 * keep ratio (keep_ratio_host[p] in (0, 1]).  Outputs, all compacted like `scores`:
 *   bitmask  [n_img, H, nb, words] uint64: bit (j % 64) of word (j / 64) set <=> query block i
 *            attends key block j; bits >= nb are zero;
 *   kept_idx [n_img, H, nb, nb] int32: the kept key blocks of row i in ascending order,
 *            entries past the count are -1;
 *   kept_cnt [n_img, H, nb] int32.
 * The comparison is done on the fp32 scores; equal scores keep the lower block index.
 */
int rapid3_select_mask(rapid3_ctx* ctx, const float* scores, const float* keep_ratio_host, int n_img,
                       uint64_t* bitmask, int32_t* kept_idx, int32_t* kept_cnt, void* stream);

/*
 * Stage (a2), threshold variant (Sec. 3.2: the sparse candidates of the policy are thresholds of
 * the sparse attention it drives, not counts; the rule itself is left to that method, so this is
 * the plain cumulative-mass rule).  Forced blocks as in rapid3_select_mask.  For the free
 * candidates c of a row, ordered by (score descending, index ascending), with weights
 *     w_c = exp(mass_scale * (S[i][c] - max over the row's free candidates)),
 * the row keeps the smallest number k >= 1 of leading candidates whose weights sum to at least
 * mass_share_host[p] * (sum of all the row's weights); a share of exactly 1 keeps all of them.
 * mass_share_host [n_img] (host) in (0, 1]; mass_scale >= 0, finite (e.g. the attention's softmax
 * scale).  The weights and their sums are fp64 on the fp32 scores; scores must be finite.
 * Outputs (device, caller-owned): row_keep [n_img, H, nb] int32 = k of every row (0 for text rows,
 * which have no free candidate), and bitmask / kept_idx / kept_cnt as in rapid3_select_mask.
 * Launches two kernels (the counts, then the selection at those counts).
 */
int rapid3_select_mask_mass(rapid3_ctx* ctx, const float* scores, const float* mass_share_host, float mass_scale,
                            int n_img, int32_t* row_keep, uint64_t* bitmask, int32_t* kept_idx,
                            int32_t* kept_cnt, void* stream);

/*
 * Stage (b): masked flash-style attention over the kept tiles only.  For image p of the list
 * (batch index img_idx_host[p], or p when the list is NULL) the kept key blocks of query block
 * i are kept_idx[p][h][i][0 .. kept_cnt[p][h][i]).  kept_idx == NULL means every block is kept
 * (dense attention) for all listed images.  Writes out[b][h][n][:] (bf16) for every token of
 * the listed images and touches nothing else.  bf16 tensor-core products, fp32 online softmax.
 * softmax_scale multiplies q.k before the softmax.
 */
int rapid3_sparse_joint_attn(rapid3_ctx* ctx, const void* q, const void* k, const void* v, void* out,
                             const int32_t* img_idx_host, int n_img, const int32_t* kept_idx,
                             const int32_t* kept_cnt, float softmax_scale, void* stream);

/*
 * One policy-gated step over a batch of B <= B_max images: action_host[b] in
 * {SKIP, REUSE, ATTEND}; only ATTEND images are processed, at keep_ratio_host[b] in (0, 1]
 * (ignored for the others).  Images with keep ratio exactly 1 skip the scoring and selection
 * passes.  Skipped and reusing images launch no work and their rows of `out` stay untouched.
 * Scores, masks and kept lists of the sparse images live in the context's workspace
 * (see rapid3_workspace), compacted in ascending batch order of the sparse images.
 * The call only launches kernels (the tensor maps of a set of base pointers are encoded on the host at
 * their first use and cached), so after one plain call with the same tensors it can be captured
 * into a CUDA graph and replayed on buffers refilled in place; the actions and ratios are then
 * those of the capture (rapid3_gated_step_device reads them on the GPU at every replay).
 */
int rapid3_gated_step(rapid3_ctx* ctx, const void* q, const void* k, const void* v, void* out,
                      const int32_t* action_host, const float* keep_ratio_host, int B,
                      float softmax_scale, void* stream);

/*
 * The same step with one keep ratio per (image, head): keep_ratio_host is [B][H], row-major
 * (Sec. 3.2: the sparsity head emits a ratio for every layer and head).  Head h of image b keeps
 * clamp(ceil(keep_ratio_host[b][h] * n_free - 1e-6)) free candidates per query-block row; forced
 * blocks are as in rapid3_select_mask.  An image whose H ratios are all exactly 1 is dense and
 * skips scoring and selection; any other attending image is scored once and selected per head.
 * Every ratio of an attending image must lie in (0, 1], else RAPID3_ERR_INVALID_ARG; the ratios of
 * gated images are ignored.  The keep counts travel as a kernel argument, so (sparse images) * H
 * may not exceed 2048: more returns RAPID3_ERR_UNSUPPORTED and launches nothing.  Workspace
 * layout and everything else are as in rapid3_gated_step.
 */
int rapid3_gated_step_heads(rapid3_ctx* ctx, const void* q, const void* k, const void* v, void* out,
                            const int32_t* action_host, const float* keep_ratio_host, int B,
                            float softmax_scale, void* stream);

/*
 * The gated step with the cumulative-mass selection of rapid3_select_mask_mass in place of the
 * top-k selection: mass_share_host[b] in (0, 1] is the share of attending image b (ignored for the
 * others); a share of exactly 1 makes the image dense (no scoring); mass_scale as in
 * rapid3_select_mask_mass.  Five launches with a sparse image (pool, scores, counts, selection,
 * attention).  The per-row counts stay in the context's workspace.  Everything else as in
 * rapid3_gated_step.
 */
int rapid3_gated_step_mass(rapid3_ctx* ctx, const void* q, const void* k, const void* v, void* out,
                           const int32_t* action_host, const float* mass_share_host, float mass_scale, int B,
                           float softmax_scale, void* stream);

/*
 * The gated step with the producer of Q and K folded in (the paper takes the block in front of the
 * attention from its base models: per-head RMS normalisation of the projected queries and keys
 * with a learned gain, then the rotary position embedding).  One kernel reads q_raw / k_raw once,
 * writes the finished bf16 q / k once and, for the images that will be scored, the block means of
 * what it wrote: the separate pooling pass over Q and K of rapid3_gated_step (the only extra HBM
 * pass the sparsity rule adds) is gone.  Per token row x[D] of an attending image:
 *     r = 1 / sqrt(mean(x^2) + eps);   y[d] = x[d] * r * gain[d];
 *     z[2i] = y[2i] cos - y[2i+1] sin,  z[2i+1] = y[2i] sin + y[2i+1] cos,  (cos, sin) = rot[n][i]
 * rounded once to bf16 (fp32 arithmetic).  Then scoring, selection and attention run on q, k, v
 * exactly as in rapid3_gated_step (4 launches with a sparse image, 2 without).
 *   q_raw, k_raw, q, k : device, bf16, the context's [B, H, N, D] strides, 16-byte aligned;
 *                        q may equal q_raw and k may equal k_raw (in place);
 *   q_gain, k_gain     : device, fp32 [D], 16-byte aligned;
 *   rot                : device, fp32 [N][D/2][2] = (cos, sin) per token and channel pair, 16-byte
 *                        aligned, or NULL for no rotation;   eps >= 0.
 * Rows of q, k and out that belong to gated images are not touched.
 */
int rapid3_gated_step_fused(rapid3_ctx* ctx, const void* q_raw, const void* k_raw, const void* v,
                            const float* q_gain, const float* k_gain, const float* rot, float eps, void* q,
                            void* k, void* out, const int32_t* action_host, const float* keep_ratio_host, int B,
                            float softmax_scale, void* stream);

/*
 * The same step with the policy's decisions left on the GPU (Sec. 3.3: the heads sample their
 * actions on the device; reading them back would cost a host synchronisation per step and layer):
 * action_dev [B] int32 and keep_ratio_dev [B] float are DEVICE arrays, read by the kernels when
 * they run on `stream`, not at call time.  A one-thread kernel builds the image lists, then the
 * four kernels of rapid3_gated_step are launched with grids sized for all B images; thread blocks
 * of images that do not attend return at once.  Results (output, workspace contents) are those of
 * rapid3_gated_step with the same actions.  An action outside {SKIP, REUSE, ATTEND} or a ratio
 * outside (0, 1] cannot be rejected at call time: that image is not processed and the device status
 * word is set to RAPID3_ERR_INVALID_ARG (see rapid3_last_status).
 */
int rapid3_gated_step_device(rapid3_ctx* ctx, const void* q, const void* k, const void* v, void* out,
                             const int32_t* action_dev, const float* keep_ratio_dev, int B,
                             float softmax_scale, void* stream);

/*
 * The same step with HOST tensors (pinned memory recommended): copies Q, K, V of the attending
 * images to device staging buffers, runs the step and copies their rows of `out` back; gated
 * images move no bytes.  The work is pipelined image by image over two copy streams owned by the
 * context (uploads of the next image, compute, downloads of the previous one overlap; the last
 * attending image goes in four groups of heads so that little is left to do after the last
 * upload), forked from and joined back into `stream`: seen from `stream` it is one ordered piece
 * of work.  The workspace afterwards describes the last piece processed only (the last head group
 * of the last attending image, with that group's head count).  The staging buffers (4 tensors of
 * B_max*H*N*D bf16, contiguous [B, H, N, D]; the host tensors must be contiguous too) are
 * allocated on the first call of a context, so make that call outside any timed region.
 * bytes_h2d / bytes_d2h (may be NULL) receive the bytes moved.
 */
int rapid3_gated_step_host(rapid3_ctx* ctx, const void* q_host, const void* k_host, const void* v_host,
                           void* out_host, const int32_t* action_host, const float* keep_ratio_host, int B,
                           float softmax_scale, void* stream, int64_t* bytes_h2d, int64_t* bytes_d2h);

/*
 * Cache-Reuse data path (Sec. 3.2 "Level-2: Cache-Reuse", the conditional definition of O_t, and
 * the cached residual Delta = G(X) - X).  x, o, delta: DEVICE bf16 arrays [B, elems_per_image],
 * contiguous, 16-byte aligned; elems_per_image a multiple of 8.  Per image b:
 *   action ATTEND: the generator has just written o[b]; the cache is refreshed, delta[b] = o[b] - x[b];
 *   action REUSE : the cached residual replaces the generator,            o[b] = x[b] + delta[b];
 *   action SKIP  : nothing is read or written.
 * The sum / difference is taken in fp32 and rounded once to bf16.  Needs no context and no
 * workspace; asynchronous on `stream`; if every image is skipped nothing is launched.
 */
int rapid3_cache_step(const void* x, void* o, void* delta, const int32_t* action_host, int B,
                      int64_t elems_per_image, void* stream);

/* Device pointers of the workspace rapid3_gated_step fills (any may be NULL): layouts as in
 * rapid3_block_scores / rapid3_select_mask with n_img = number of sparse images of the last step. */
int rapid3_workspace(rapid3_ctx* ctx, float** scores, uint64_t** bitmask, int32_t** kept_idx,
                     int32_t** kept_cnt);

/* Number of kernels this context has launched so far (all entry points). */
int64_t rapid3_launch_count(rapid3_ctx* ctx);

/*
 * Measurement aid (no counterpart in the paper): with profiling enabled (enable = 1) every kernel
 * launch of this context is bracketed by a CUDA event pair on the caller's stream (at most 16384
 * pairs between reads); enable = 2 brackets the attention kernel only (an event pair costs a few
 * microseconds of stream time, which matters beside the short scoring kernels); 0 switches it off.  rapid3_profile_read waits for the recorded events, returns the summed device
 * time in milliseconds and the launch count per kernel kind
 * (0 block pool, 1 block scores, 2 mask select, 3 attention) and clears the record.
 */
int rapid3_profile(rapid3_ctx* ctx, int enable);
int rapid3_profile_read(rapid3_ctx* ctx, double* ms /* [4] */, int64_t* launches /* [4] */);

/*
 * Scoring pass without any allocation (the paper has no counterpart; this exists for the callers
 * described here).  rapid3_create obtains the workspace with cudaMalloc.  Some hosts of this
 * library cannot do that: an inference server whose own allocator has already reserved all of
 * the GPU's memory (a later cudaMalloc from a plug-in fails), or a latency-critical sampling loop
 * that must not take the device-wide synchronisation an allocation implies.  For them this
 * entry point computes exactly what rapid3_block_scores computes -- scores[p][h][i][j], fp32,
 * [n_img, H, nb, nb], same kernels, same rounding -- without a context: the block means go to a
 * fixed array inside the library's device image instead of an allocated workspace.
 *
 *   - `shape` describes Q and K as for rapid3_create (B_max only bounds the batch indices).
 *   - Limit: 2 * n_img * H * nb * D block means (fp64) must fit rapid3_static_scratch_bytes()
 *     = 16 MiB, e.g. four FLUX 1024^2 images (24 heads, D = 128, 72 blocks) or one FLUX 2048^2
 *     image per call; a larger request returns RAPID3_ERR_WORKSPACE and launches nothing.
 *     Every GPU that loads the library holds these 16 MiB until the process exits.
 *   - The first call on a device looks up the array's device address (once per device, with
 *     that device current); make that first call before starting any stream capture.
 *   - Calls no cudaMalloc / cudaFree and no allocating library routine; asynchronous on `stream`.
 *   - All calls on a device share the one array and it keeps the previous call's contents.
 *     Nothing in it has to start at zero (the pooling kernel writes every element the scoring
 *     kernel reads), but two calls that overlap on the GPU (different streams, no dependency)
 *     race on it: order them on one stream or with events.
 */
int rapid3_block_scores_static(const rapid3_shape* shape, const void* q, const void* k,
                               const int32_t* img_idx_host, int n_img, float* scores, void* stream);
/* Size in bytes of the fixed scratch array of rapid3_block_scores_static. */
int64_t rapid3_static_scratch_bytes(void);

/*
 * Cost report of one sampling trajectory (Sec. 3.3, "equivalent steps"): host arithmetic only.
 *   K = sum over the steps that run of (1 - C_cache[k]) * (1 - C_sparse[k]),
 * where C_cache[k] is the cost reduction of a step that reuses the cache and C_sparse[k] that of a
 * step that attends sparsely, both in [0, 1].  action_host[k] says what step k did: a SKIP step
 * does not run and adds nothing; a REUSE step adds 1 - c_cache_host[k] (it runs no attention, so
 * no sparse reduction applies); an ATTEND step adds 1 - c_sparse_host[k] (0 for dense attention).
 * *k_exact (may be NULL) receives the sum in fp64, *k_rounded (may be NULL) the nearest integer,
 * halves upward.  n_steps >= 0.  A reduction outside [0, 1] or an unknown action returns
 * RAPID3_ERR_INVALID_ARG and writes nothing.  No GPU work, no context.
 */
int rapid3_equivalent_steps(const int32_t* action_host, const float* c_cache_host, const float* c_sparse_host,
                            int n_steps, double* k_exact, int64_t* k_rounded);

/* Copies the device status word to *device_status (RAPID3_OK or a negative code) and clears it.
 * Synchronises the device; call it after the stream has been synchronised. */
int rapid3_last_status(rapid3_ctx* ctx, int* device_status);

/*
 * Test aid for the failure path (no counterpart in the paper; not part of the hot path).
 * Launches a separately compiled failure-injection build of the attention kernel as a dense
 * attention over image 0 of q, k, v: its producer stops issuing copies before group `stop_group`
 * (group g = key block g together with value block g - 1; 0 <= stop_group <= nb), and every
 * barrier wait in it gives up after 4096 polls instead of 2^22.  The waits of the other roles
 * therefore run out: each thread block records RAPID3_ERR_TIMEOUT in the status word, waits
 * (bounded) for its copies in flight, lets its tensor-core work finish, releases its tensor
 * memory and returns.  Nothing waits without a limit and nothing faults; `out` is left partly
 * or wholly unwritten.  The context stays usable: after rapid3_last_status has returned (and
 * cleared) the code, ordinary calls compute as before.  Asynchronous on `stream`.
 */
int rapid3_debug_inject_timeout(rapid3_ctx* ctx, const void* q, const void* k, const void* v, void* out,
                                int stop_group, float softmax_scale, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RAPID3_H_ */
