/*
 * scalekv.h - C ABI of the ScaleKV per-scale hot path for NVIDIA B200 (sm_100a).
 *
 * The library implements, with hand-written CUDA kernels, the step that scale-aware KV-cache
 * compression (arXiv 2505.19602) adds to next-scale-prediction inference: for every scale k of
 * the coarse-to-fine schedule and every transformer layer l,
 *
 *     append   : the K/V rows of the current token map r_k join the layer's cache, so that the
 *                keys are P_{k-1} U C_k                                  (Sec. 1; Sec. 3.3, ASI paragraph)
 *     attend   : O = softmax(Q K^T / sqrt(d)) V over every cache entry   (Sec. 3.3, Eq. 5)
 *     compress : observation-window scores, top-k^l selection, pruning   (Sec. 3.3, "KV Cache Selection")
 *
 * plus the offline statistics that split layers into drafters and refiners (Sec. 3.3, Eq. 2-4).
 *
 * Conventions
 *  - A "slice" is one (layer, batch, head) triple; slices never exchange data.
 *  - Every function returns a scalekv_status.  Argument and call-order errors are reported
 *    synchronously and leave the device untouched.  Device-side errors (a bounded wait that gave
 *    up, a failed bounds check) are recorded in a sticky status word and returned by scalekv_sync.
 *  - append / attend / compress only enqueue work on the caller's CUDA streams and return.
 *  - Ownership: the caller owns the pool, the workspace, the streams and every tensor it passes.
 *    The library owns only the host-side context.  It never allocates device memory after
 *    scalekv_init and never falls back to the CPU: an unsupported (dtype, head_dim) pair is an error.
 *  - Pointers are DEVICE pointers unless a parameter is documented as HOST.
 *  - One context must be used by one host thread at a time.
 */
#ifndef SCALEKV_H
#define SCALEKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct scalekv_ctx scalekv_ctx; /* opaque, host-side, library-owned */

typedef enum {
  SCALEKV_OK = 0,
  SCALEKV_ERR_INVALID_ARG = 1,  /* null pointer, size out of range, misaligned tensor            */
  SCALEKV_ERR_BAD_STATE = 2,    /* call out of order for this layer (append -> attend -> compress) */
  SCALEKV_ERR_CAPACITY = 3,     /* pool or workspace smaller than scalekv_query_sizes reports     */
  SCALEKV_ERR_UNSUPPORTED = 4,  /* (dtype, head_dim) not built: bf16 x 128 and f32 x 64 are        */
  SCALEKV_ERR_CUDA = 5,         /* a CUDA runtime/driver call failed; text in scalekv_error_string */
  SCALEKV_ERR_TIMEOUT = 6,      /* a bounded device-side wait gave up (reported by scalekv_sync)   */
  SCALEKV_ERR_DEVICE_CHECK = 7  /* a device-side bounds check tripped (reported by scalekv_sync)   */
} scalekv_status;

typedef enum { SCALEKV_BF16 = 0, SCALEKV_F32 = 1 } scalekv_dtype;

#define SCALEKV_KEEP_ALL (-1)   /* budget value: never evict                                       */
#define SCALEKV_MAX_WINDOW 64   /* largest explicit observation window (a whole-map window is free) */
#define SCALEKV_MAX_SCALES 32

typedef struct {
  int32_t n_layers, batch, n_heads, head_dim;
  int32_t dtype;                 /* scalekv_dtype of Q, K, V, O and of the cache                    */
  int32_t n_scales;
  const int32_t *scale_h;        /* HOST [n_scales]: token-map heights h_k (copied)                 */
  const int32_t *scale_w;        /* HOST [n_scales]: token-map widths  w_k (copied)                 */
  const int32_t *budgets;        /* HOST [n_layers][n_scales]: k^l of the compress issued during    */
                                 /* scale k = number of NON-window entries kept; SCALEKV_KEEP_ALL   */
                                 /* or any value >= the candidates means no eviction (copied)       */
  int32_t max_window;            /* upper bound on the explicit window size w, <= SCALEKV_MAX_WINDOW */
  float softmax_scale;           /* 0 => 1/sqrt(head_dim) (Eq. 5)                                   */
  int32_t page_tokens;           /* tokens per page; 0 => 128; must be a power of two >= 16         */
  void *pool;                    /* device memory for pages, page tables and lengths (borrowed)     */
  size_t pool_bytes;
  void *workspace;               /* device scratch for scores, keep lists, statistics (borrowed)    */
  size_t workspace_bytes;
  void *stream_main;             /* cudaStream_t: append and attend run here                        */
  void *stream_side;             /* cudaStream_t: compress runs here (may equal stream_main)        */
  int32_t device;                /* CUDA device ordinal that owns pool, workspace and streams       */
  int32_t window_patches;        /* N of Sec. 3.3 (e.g. 16), or 0.  When > 0, scalekv_attend (bf16 x 128)  */
                                 /* also records the logits of the N-patch centroid rows of the current */
                                 /* map (scalekv_window_centroids) while it computes them anyway, and a */
                                 /* scalekv_compress called with exactly that window scores the cache   */
                                 /* from them instead of reading K again.  Any other window still works.*/
                                 /* Nothing is recorded at the last scale of the schedule (nothing is      */
                                 /* generated after it, so the method prunes nothing there) nor by a        */
                                 /* scalekv_step that names no window: a compress then scores from K.       */
  int32_t window_kind;           /* which rows window_patches = N stands for: SCALEKV_WINDOW_CENTROIDS (0, the   */
                                 /* paper's patch centroids) or SCALEKV_WINDOW_LAST (the last N rows of the map */
                                 /* in raster order, scalekv_window_last - the SnapKV-like comparison rule)     */
} scalekv_config;
#define SCALEKV_WINDOW_CENTROIDS 0
#define SCALEKV_WINDOW_LAST 1

/* A [batch][n_heads][tokens][head_dim] tensor view: device pointer + ELEMENT strides; the
 * innermost (head_dim) axis is contiguous and every row must start on a 16-byte boundary. */
typedef struct {
  const void *ptr;
  int64_t stride_b, stride_h, stride_t;
} scalekv_tensor;

/* ---- life cycle ------------------------------------------------------------------------- */

/* Bytes of pool and workspace that scalekv_init needs for this configuration (pointers in cfg
 * are ignored).  The pool holds, per layer, ceil(cap_l / page_tokens) persistent pages per slice,
 * cap_l being the largest cache a compress leaves behind, plus four transient page sets (layer l
 * uses set l mod 4) that hold the part of the current map that exceeds cap_l until that layer's
 * compress; page tables; per-slice lengths.  No CUDA call is made. */
scalekv_status scalekv_query_sizes(const scalekv_config *cfg, size_t *pool_bytes, size_t *workspace_bytes);

/* Creates a context: copies schedule and budgets, carves the pool, uploads the page tables and
 * zeroes the lengths (synchronous).  *out is NULL on failure. */
scalekv_status scalekv_init(const scalekv_config *cfg, scalekv_ctx **out);

/* Empties every slice (start of a new image batch).  Enqueued on stream_main after both streams'
 * pending work.  The hot calls only enqueue kernels, memsets and event fork/joins between the two
 * streams, so a sequence reset, {append, attend, compress}... can be captured on stream_main into a
 * CUDA graph and replayed (call scalekv_join before ending the capture). */
scalekv_status scalekv_reset(scalekv_ctx *ctx);

/* Makes stream_main wait for everything enqueued so far on stream_side.  Only enqueues an event record
 * and a wait: legal during a capture. */
scalekv_status scalekv_join(scalekv_ctx *ctx);

/* Waits for both streams and frees the host context.  Device memory stays with the caller. */
scalekv_status scalekv_destroy(scalekv_ctx *ctx);

/* ---- the hot path ------------------------------------------------------------------------ */

/* Sec. 1 / Sec. 3.3: the current map joins the cache.  K and V are [B][H][n_k][d] views of the
 * n_k = h_k * w_k rows of scale `scale` (0-based; scales must arrive in ascending order, once per
 * layer).  Row i receives original position N_{k-1} + i.  The rows are copied into the store.
 * For bf16 x 128 the copy is done by the scalekv_attend that follows, which reads the map from K
 * and V directly and writes its rows to the pages while it streams them (no second read, nothing
 * on the critical path); any other next call for this layer (compress, layer_stats, export, the
 * next append) copies first with a kernel of its own.  K and V must therefore stay unmodified
 * until stream_main has passed the layer's next call.  For f32 x 64 the copy is enqueued here.
 * Ordered on stream_main after this layer's previous compress.
 * Layers l, l + 4, l + 8, .. share one transient page set, which holds the part of a
 * current map that exceeds the layer's persistent capacity, and one buffer of recorded window logits.  An append
 * therefore returns SCALEKV_ERR_BAD_STATE, and touches nothing, while another layer of the same set still
 * holds an appended map that reaches into the transient pages and has not been compressed; otherwise it waits
 * (on stream_main) for that layer's last compress.  The one exception is a map of the LAST scale that has been
 * attended: no later step reads it, so its transient rows are given up, and that layer then refuses compress and
 * layer_stats (BAD_STATE) and exports only the entries before that map until scalekv_reset.  The model's own order -
 * append, attend, compress of layer l before layer l + 1 - never meets this rule. */
scalekv_status scalekv_append(scalekv_ctx *ctx, int32_t layer, int32_t scale, scalekv_tensor K, scalekv_tensor V);

/* Eq. 5: O[b][h][i] = sum_j softmax_j(scale * <Q[b][h][i], K_j>) V_j over all L entries of the
 * slice (history that survived earlier compressions, then the current map).  Q and O are
 * [B][H][n_k][d] views in the configured dtype; lse (nullable) is a dense float [B][H][n_k]
 * that receives max + log-sum-exp of the scaled logits.  bf16: products are exact, sums are
 * fp32, P is rounded to bf16 before the PV product.  f32: plain fp32 FMA.  Runs on stream_main. */
scalekv_status scalekv_attend(scalekv_ctx *ctx, int32_t layer, scalekv_tensor Q, scalekv_tensor O, float *lse);

/* Sec. 3.3 "KV Cache Selection": with A = softmax(Q_W K^T * scale) over all L entries,
 * s_i = (1/w) sum_{j in W} A_ji (Eq. 5, mean over the window rows, per head, fp32); the
 * candidates are all entries that are not window entries; the k' = min(k^l, #candidates) best are
 * kept (equal scores: lowest original position first) together with the w window entries; the
 * survivors are moved to the front of the slice in ascending original position, in place.
 *   Qw          window queries.  qw_is_full_map == 0: a [B][H][w][d] view whose row j is the query
 *               at window_pos[j].  qw_is_full_map != 0: the [B][H][n_k][d] query tensor of the
 *               current map; the library reads rows window_pos[j] itself.
 *   w           window size, 1 <= w <= max_window; ignored when window_pos is NULL.
 *   window_pos  HOST array [w] of distinct raster indices (r * w_k + c) inside the current map,
 *               ascending, identical for every slice.  NULL means the window is the whole current
 *               map (w = n_k; requires n_k <= SCALEKV_MAX_WINDOW and a dense Qw of n_k rows).
 * k^l is budgets[layer][scale] of the scale last appended.  If nothing can be evicted the call
 * only commits the lengths.  Runs on stream_side after this layer's attend. */
scalekv_status scalekv_compress(scalekv_ctx *ctx, int32_t layer, scalekv_tensor Qw, int32_t w,
                                const int32_t *window_pos, int32_t qw_is_full_map);

/* Variants of the selection rule (the readings and comparison policies the paper names beside its own).
 *   policy       SCALEKV_SELECT_SCORE: the observation-window importance of Sec. 3.3 (scalekv_compress).
 *                SCALEKV_SELECT_RECENT: positional, as in the comparison policies of Sec. 4.1 (sliding
 *                window; attention sinks + recent tokens): there is no observation window (Qw, w,
 *                window_pos are ignored), the n_sink lowest original positions always stay and the most
 *                recent other entries fill the budget; here k^l = budgets[layer][scale] counts the WHOLE
 *                cache after the call, sinks included.  The layer's pages were sized from the table, so
 *                min(n_sink, tokens so far) beyond the persistent capacity returns SCALEKV_ERR_CAPACITY.
 *   pool_kernel  SCORE only.  Odd width (< 64) of a 1-D average pooling of the importance along the slot
 *                axis before the selection ("average pooling", Sec. 3.3, read as smoothing along keys: zeros
 *                beyond both ends, always divided by the width; the neighbours are the entries next to it in
 *                the cache as it stands, window entries included).  0 or 1: none - the default reading.
 *   head_shared  SCORE only.  1: one importance for all heads of a batch element ("a unified importance
 *                metric", Sec. 3.3, read as shared between heads): the mean over the heads of the per-head
 *                importance, entry by entry, taken before the pooling; every head then keeps the same
 *                entries.  Needs the heads of a batch element to hold the same original positions, which is
 *                the case when the layer was compressed this way from its first scale on; otherwise the
 *                device status turns to SCALEKV_ERR_DEVICE_CHECK (reported by scalekv_sync, sticky) and
 *                neither the selection nor the compaction runs.
 *                0: per head - the default reading.  At most 256 heads.
 *   head_budgets HOST array [n_heads] or NULL.  Budgets of this call per head (the same for every batch
 *                element) in place of budgets[layer][scale]: the store is ragged, so heads may keep
 *                different numbers of entries.  Each value must lie in [0, budgets[layer][scale]] (the
 *                pages were sized for the table's value); any value >= 0 when the table says KEEP_ALL.
 *                With head_shared the heads must agree.  At most 128 heads.
 *   separate_kernels  0: importance, selection and pruning of a slice run in ONE launch (one CTA per slice, the
 *                slice's keys and keep list in shared memory) whenever a slice of the configured schedule fits;
 *                1: as three launches (importance; selection; pruning spread over 8 CTAs per slice), which is what
 *                slices too long for one CTA's shared memory and head_shared get in any case.  Same results.
 * opts == NULL is scalekv_compress. */
#define SCALEKV_SELECT_SCORE 0
#define SCALEKV_SELECT_RECENT 1
typedef struct {
  int32_t policy;
  int32_t pool_kernel;
  int32_t n_sink;        /* RECENT only */
  int32_t head_shared;   /* SCORE only */
  const int32_t *head_budgets;
  int32_t separate_kernels;   /* see below */
} scalekv_select_opts;
scalekv_status scalekv_compress_ex(scalekv_ctx *ctx, int32_t layer, scalekv_tensor Qw, int32_t w, const int32_t *window_pos,
                                   int32_t qw_is_full_map, const scalekv_select_opts *opts);

/* One whole step for one layer from DEVICE tensors, in one call: scalekv_append(K, V), scalekv_attend(Q -> O
 * [, lse]) and, with the window rows taken from Q (the full current map), scalekv_compress.
 * w > 0: window_pos holds w raster indices; w < 0: the whole current map is the window; w == 0: no
 * compress.  Same results as the three calls; saves two trips through the binding per step.
 * Because the step knows what follows its attend, it does not write rows into the store that nothing will read: when
 * its compress evicts, the attend leaves the current map in K and V and the compress (on stream_side) takes the
 * surviving rows from there - in a layer with a 3 % budget 19 of 20 rows of a map would otherwise be written only to
 * be dropped; after the last scale with w == 0 the map stays in K and V until a later call for the layer (export,
 * layer_stats) copies it, if one comes.  K and V (and Q, which the compress may read) must therefore stay unmodified
 * until the step's compress has completed: until stream_main has passed the layer's next append, or scalekv_join or
 * scalekv_sync; after the last scale, until the layer's next call has passed on stream_main or scalekv_reset. */
scalekv_status scalekv_step(scalekv_ctx *ctx, int32_t layer, int32_t scale, scalekv_tensor Q, scalekv_tensor K,
                            scalekv_tensor V, scalekv_tensor O, float *lse, int32_t w, const int32_t *window_pos);

/* scalekv_step with a selection variant: compress == 0: no compress; otherwise the step ends with
 * scalekv_compress_ex(layer, Q as the full current map, w, window_pos, opts) - Sec. 4.1's comparison rules as one-call
 * steps (w and window_pos as scalekv_compress_ex takes them: ignored by SCALEKV_SELECT_RECENT, window_pos == NULL for the
 * whole map).  Same results and the same contract as scalekv_step. */
scalekv_status scalekv_step_ex(scalekv_ctx *ctx, int32_t layer, int32_t scale, scalekv_tensor Q, scalekv_tensor K,
                               scalekv_tensor V, scalekv_tensor O, float *lse, int32_t compress, int32_t w,
                               const int32_t *window_pos, const scalekv_select_opts *opts);

/* One whole step for one layer from HOST memory (pinned memory recommended): copies Q, K, V
 * (dense [B][H][n_k][d]) to `staging`, runs append, attend and compress with the window rows
 * taken from Q (w > 0: explicit window_pos; w < 0: the whole map is the window; w == 0: no
 * compress), and copies O back to O_host.  staging is device memory of at least
 * 8 * B*H*n_k*d elements: consecutive calls alternate between its two halves, and the copies run
 * on two streams of the library's own (created at the first call), so that a step's input copy, the
 * previous step's kernels and the output copy before that overlap.  Everything is enqueued; the
 * host buffers must stay valid, and O_host is complete, once scalekv_sync has returned. */
scalekv_status scalekv_step_host(scalekv_ctx *ctx, int32_t layer, int32_t scale, const void *Q_host,
                                 const void *K_host, const void *V_host, void *O_host, void *staging,
                                 size_t staging_bytes, int32_t w, const int32_t *window_pos);

/* ---- offline statistics and host-side policy (Sec. 3.3, Eq. 2-4) --------------------------- */

/* Eq. 2 for the scale last appended to `layer` (call after append, cache uncompressed): for every
 * query row i = 0, query_stride, 2*query_stride, ... of Q and every slice, alpha_i = softmax row
 * over all entries; c_i = mass on the current map; t_i = sum of the min(K', |history|) largest
 * alpha_ij over the history.  *car and *htk (HOST) receive the means of c_i and t_i over rows and
 * slices; ASI = car * htk.  Synchronous; not part of the timed path.  topk_prime <= 64. */
scalekv_status scalekv_layer_stats(scalekv_ctx *ctx, int32_t layer, scalekv_tensor Q, int32_t topk_prime,
                                   int32_t query_stride, double *car, double *htk);

/* The same statistics, also per slice.  car_slices / htk_slices (HOST, [batch * n_heads], either may be
 * NULL) receive the means of c_i and t_i over the sampled rows of each slice.  nca_slices (HOST,
 * [batch * n_heads] or NULL) receives the "normalized current scale attention" of Sec. 4.3 per slice:
 * the average attention a query gives to one token of the current map, c_i / n_k, over the average
 * it gives to one entry of the whole sequence, 1 / L, averaged over the sampled rows, i.e.
 * car_slice * L / n_k with L the slice's length (the distribution the paper plots over scales). */
scalekv_status scalekv_layer_stats_ex(scalekv_ctx *ctx, int32_t layer, scalekv_tensor Q, int32_t topk_prime,
                                      int32_t query_stride, double *car, double *htk, double *car_slices,
                                      double *htk_slices, double *nca_slices);

/* Sec. 3.3: the observation window = centroid token of each of N patches of an h x w map.
 * g = floor(sqrt(N)) patches per side, patch (a,b) = rows [a*h/g, (a+1)*h/g) x cols alike, centroid =
 * lower-middle cell; a map with at most N tokens is its own window.  pos (HOST, room for N entries)
 * receives ascending raster indices, *count their number.  Host only. */
scalekv_status scalekv_window_centroids(int32_t h, int32_t w, int32_t n_patches, int32_t *pos, int32_t *count);

/* Eq. 3: Z = (ASI - mu_k) / (sigma_k + eps) per scale over layers (population sigma); drafters are
 * the pairs with the lowest Z.  asi HOST [L][K] row-major.  mode 0: the n_drafters lowest pairs over
 * all ranked (layer, scale) pairs; mode 1: the n_drafters lowest layers at every ranked scale.
 * Scales 0 and K-1 are not ranked (no history / nothing follows).  Ties: lower scale, then lower
 * layer.  is_drafter HOST [L][K] receives 0/1.  Host only. */
scalekv_status scalekv_assign_roles(const double *asi, int32_t L, int32_t K, int32_t n_drafters, int32_t mode,
                                    double eps, uint8_t *is_drafter);

/* Eq. 4: B_r(k) = max(B_r(0) - delta * k, 0) for k = 1..K; per scale N_d^k B_d(k) + N_r^k B_r(k) =
 * B_uniform * L, which sums to the printed constraint; a scale without drafters gets B_uniform
 * everywhere; values rounded half up.  budgets_out HOST [L][K].  Host only. */
scalekv_status scalekv_make_budgets(const uint8_t *is_drafter, int32_t L, int32_t K, double b_uniform, double b_r0,
                                    double delta, int32_t *budgets_out);

/* Sec. 4.1 "Compression Baselines": the comparison policies as configurations of this store (their image
 * quality is outside this library; they run on the same cache for A/B timing):
 *   sliding window        SCALEKV_SELECT_RECENT, n_sink = 0, a uniform table
 *   sinks + recent tokens SCALEKV_SELECT_RECENT, n_sink > 0, a uniform table
 *   SnapKV-like           SCALEKV_SELECT_SCORE observed by the LAST rows of the map (scalekv_window_last,
 *                         window_kind = SCALEKV_WINDOW_LAST), importance pooled along the keys (pool_kernel, e.g.
 *                         7), a uniform table
 *   pyramid budgets       the SnapKV-like rule with a table that falls linearly with the layer index.
 * scalekv_window_last: the last min(n_obs, h * w) raster indices of an h x w map, ascending -> pos (HOST, room
 * for n_obs entries), *count their number.
 * scalekv_policy_budgets: budgets_out HOST [L][K], every scale alike.  SCALEKV_BUDGETS_UNIFORM: b_mean rounded
 * half up everywhere.  SCALEKV_BUDGETS_PYRAMID: layer l gets b_max - (b_max - b_min) l / (L - 1) rounded half
 * up, with b_min = b_mean / beta (beta >= 1) and b_max = 2 b_mean - b_min, so the mean over layers is b_mean;
 * a single layer gets b_mean.  Host only. */
#define SCALEKV_BUDGETS_UNIFORM 0
#define SCALEKV_BUDGETS_PYRAMID 1
scalekv_status scalekv_window_last(int32_t h, int32_t w, int32_t n_obs, int32_t *pos, int32_t *count);
scalekv_status scalekv_policy_budgets(int32_t shape, int32_t L, int32_t K, double b_mean, double beta, int32_t *budgets_out);

/* Sec. 4.1 / Sec. 4.3: a budget quoted as a fraction of "the original KV cache size" is that fraction of
 * T_c = N_{K-1}, the tokens that ever need caching (the last map is never read by a later step - Table 1's
 * full-cache sizes divide by exactly that count), rounded half up: *tokens = floor(fraction * T_c + 1/2).
 * 13-scale schedule: 0.30 -> 1928, 0.03 -> 193, 0.10 -> 643.  Host only. */
scalekv_status scalekv_budget_tokens(double fraction, const int32_t *scale_h, const int32_t *scale_w, int32_t n_scales,
                                     int32_t *tokens);

/* ---- introspection ------------------------------------------------------------------------ */

/* Current number of entries of every slice of a layer -> len_host HOST [B][H].  Synchronous. */
scalekv_status scalekv_lengths(scalekv_ctx *ctx, int32_t layer, int32_t *len_host);

/* Copies one slice to the host: original positions (pos_host [cap]), and, if non-NULL, its K and V
 * rows ([cap][d] in the configured dtype).  *len receives the entry count; fails with CAPACITY if it
 * exceeds cap.  Synchronous.  Rows beyond the layer's persistent capacity live in pages shared with
 * other layers and are only meaningful until the layer after next appends. */
scalekv_status scalekv_export_slice(scalekv_ctx *ctx, int32_t layer, int32_t b, int32_t h, int32_t *pos_host,
                                    void *K_host, void *V_host, int32_t cap, int32_t *len);

/* Importance scores of one slice as left by the most recent evicting compress (any layer):
 * s_host HOST [cap] floats indexed by the slot order BEFORE that compress.  Synchronous. */
scalekv_status scalekv_export_scores(scalekv_ctx *ctx, int32_t b, int32_t h, float *s_host, int32_t cap, int32_t *len);

/* Waits for both streams; returns the sticky device status (OK, TIMEOUT or DEVICE_CHECK). */
scalekv_status scalekv_sync(scalekv_ctx *ctx);

/* Self-test of the failure path every device-side wait of the library shares (no counterpart in the paper).
 * A one-CTA kernel waits, through the same bounded-wait routine the attention kernel uses, on a barrier
 * that nothing ever arrives at, with a limit of limit_ms (1 .. 1000) instead of the library's 2 s.  The wait
 * gives up after the limit, raises the sticky device status and the kernel RETURNS (it never spins without
 * bound, traps or faults).  *gave_up (HOST) = 1 when the wait reported the time-out, *seen_by_peer (HOST) = 1
 * when a second warp of the CTA saw the CTA-wide abort flag that the give-up sets.  Synchronous on
 * stream_main.  Afterwards scalekv_sync returns SCALEKV_ERR_TIMEOUT and every later attention CTA returns at
 * once (the status is sticky for the context's life): use a context of its own. */
scalekv_status scalekv_selftest_wait(scalekv_ctx *ctx, int32_t limit_ms, int32_t *gave_up, int32_t *seen_by_peer);

/* Number of kernels this context has launched since scalekv_init (HOST out). */
scalekv_status scalekv_launch_count(scalekv_ctx *ctx, int64_t *count);

/* Per-kernel-class device timing.  on = 1: every launch is bracketed by CUDA events on the stream
 * it runs on (durations of kernels on the two streams may overlap and then include contention).
 * on = 2: compress runs on stream_main as well, so that no two kernels overlap and each duration
 * is the kernel's own.  on = 0: off.  scalekv_profile_read waits for both streams and returns, for
 * class `which` (0 append, 1 attend, 2 score, 3 select, 4 compact, 5 other, 6 compress = importance, selection
 * and pruning in one launch), the
 * summed milliseconds and the number of launches since profiling was last enabled. */
scalekv_status scalekv_profile_enable(scalekv_ctx *ctx, int32_t on);
scalekv_status scalekv_profile_read(scalekv_ctx *ctx, int32_t which, double *ms_total, int64_t *launches);

/* ---- allocation-free top-k ------------------------------------------------------------------ */

/* (The paper has no counterpart of this call; it exists for integration reasons only.)
 * Some hosts of this library may not allocate device memory at the point where they need a
 * selection: an inference engine that sized every buffer at start-up and has handed the rest of
 * the GPU to its own pool, or code running in a phase where an allocation (cudaMalloc
 * synchronises the whole device) would stall concurrent work.  scalekv_select_static serves
 * them: it needs no context, no pool and no workspace.  The keys of its radix select live in a
 * fixed array inside the library image, so the call allocates nothing - no cudaMalloc, no
 * cudaFree, no allocating library routine.
 *
 *   scores   device, n_rows rows of `len` non-negative finite floats, row stride `ld` (>= len)
 *   k        1 <= k <= len: how many entries of each row to select
 *   idx_out  device, [n_rows][k] int32: the ascending indices of each row's k largest scores;
 *            equal scores are taken lowest index first (the rule of scalekv_compress)
 *   stream   cudaStream_t of the CURRENT device; the kernel is enqueued there, the call returns
 *
 * Limit: n_rows * len <= SCALEKV_SELECT_STATIC_MAX_ENTRIES (4 MiB of keys); larger requests
 * return SCALEKV_ERR_CAPACITY and print the reason to stderr.  Every device that loads the
 * library holds this array until the process ends.
 * The first call on each device looks up the array's device address (once, under a lock);
 * make that first call before starting any stream capture on that device.
 * All calls on a device share the one array and find in it whatever the previous call left;
 * nothing in it has to start at zero, because every call first overwrites the keys it reads.
 * Two calls whose kernels may overlap on the GPU (different streams, no ordering) race on it:
 * order them on one stream or with events. */
#define SCALEKV_SELECT_STATIC_MAX_ENTRIES (1 << 20)
scalekv_status scalekv_select_static(const float *scores, int32_t n_rows, int32_t len, int32_t ld, int32_t k,
                                     int32_t *idx_out, void *stream);

/* Text of the last error of this context (never NULL; valid until the next call). */
const char *scalekv_error_string(scalekv_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* SCALEKV_H */
