/* purekv.h -- C ABI of the PureKV hot path for NVIDIA B200 (sm_100a).
 *
 * The library implements, as hand-written CUDA kernels, the data-parallel part of
 * PureKV: Spatial-Temporal Sparse Attention (ST-SpAttn) prefill (Sec. 3.2) and the
 * KV-cache compression it feeds (Sec. 3.1): window attention scores of a low layer
 * (Eq. 1-2), V-norm weighting (Eq. 3-4), selection of the recent window plus the
 * top-h non-recent keys, and the gather of the surviving K/V rows.
 *
 * Conventions
 *  - Every function returns a purekv_status; nothing throws across the ABI.
 *  - The caller owns every buffer.  Pointers are DEVICE pointers unless the name
 *    starts with h_ (host).  Nothing is allocated or freed by the library, and no
 *    call synchronises the device unless its comment says so.
 *  - `stream` is a cudaStream_t passed as void*; all device work is enqueued on it.
 *  - Packed variable-length layout ("THD"): Q and O are [T, H, d], K and V are
 *    [T, H_kv, d], row-major, contiguous; T = total tokens over all requests and
 *    request r owns tokens cu_seqlens[r] .. cu_seqlens[r+1]-1.  Query head hq uses KV
 *    head hq / (H / H_kv).
 *  - A request's tokens are ordered [n_prefix text][n_frames x (grid_h x grid_w) visual,
 *    raster order inside a frame][suffix text].
 *  - dtype is the element type of Q/K/V/O; accumulation, softmax and scores are fp32.
 *  - A batch with no requests or no tokens is valid everywhere: the call returns PUREKV_OK
 *    without touching any buffer (tensor pointers may then be null).
 */
#ifndef PUREKV_H_
#define PUREKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  PUREKV_OK = 0,
  PUREKV_ERR_INVALID_ARG = 1, /* null pointer, negative size, inconsistent descriptors   */
  PUREKV_ERR_UNSUPPORTED = 2, /* head_dim / dtype / tile combination without a kernel    */
  PUREKV_ERR_WORKSPACE = 3,   /* plan or workspace buffer too small                      */
  PUREKV_ERR_CUDA = 4,        /* a CUDA call failed; text in purekv_last_error           */
  PUREKV_ERR_TIMEOUT = 5,     /* a bounded device-side wait expired (purekv_poll_status) */
  PUREKV_ERR_BAD_PLAN = 6     /* a kernel found the plan it was handed inconsistent and did not use it (purekv_poll_status) */
} purekv_status;

typedef enum { PUREKV_BF16 = 0, PUREKV_FP32 = 1 } purekv_dtype;

#define PUREKV_FLAG_DENSE_CAUSAL 1u
#define PUREKV_FLAG_COARSE_BLOCKS 2u

/* The ST-SpAttn mask (Sec. 3.2).  The paper's mask is {anchor_frames 1, spatial_radius -1,
 * temporal_depth 1, temporal_stride 1, temporal_radius 0}: a visual query attends the first
 * frame, its own frame, and its own grid cell in the previous frame, all under causality.
 * Other values are this library's extension.  Text queries are dense causal and prefix keys
 * are visible to every query.  The mask is token-exact; `tile` only sets the granularity at
 * which fully masked key blocks are skipped -- unless PUREKV_FLAG_COARSE_BLOCKS is set: then the
 * mask is widened to tile x tile blocks of request positions (a block pair is kept whole, under
 * causality, as soon as it holds one kept pair), the block-sparse reading of the same mask.
 * The sparse-attention variants the paper compares with (App. A.3, Table 7; the paper names
 * them and shows them in a figure only, so the settings are the usual meanings of the names):
 *   Spatial Sparse Attention   {1, -1, 0, 1, 0}: the spatial path alone, first frame + own frame;
 *   Temporal Sparse Attention  {1,  0, 1, 1, 0}: the temporal path alone, first frame + own cell
 *                              of the previous frame (+ the token itself);
 *   Local Attention            {0,  0, 0, 1, 0} with local_window = L: the L most recent positions;
 *   Atrous Attention           {0,  0, 0, 1, 0} with atrous_dilation = D: every D-th earlier position.
 * A visual query sees the union of whatever terms are switched on. */
typedef struct {
  int32_t grid_h, grid_w;  /* per-frame token grid                                         */
  int32_t anchor_frames;   /* first frames every visual query sees                         */
  int32_t spatial_radius;  /* -1: whole current frame; else Chebyshev radius in the grid   */
  int32_t temporal_depth;  /* number of linked earlier frames; -1: all                     */
  int32_t temporal_stride; /* linked frames are f-s, f-2s, ... (>= 1)                      */
  int32_t temporal_radius; /* 0: same grid cell; r: Chebyshev radius; -1: whole frame      */
  int32_t tile;            /* key-block size for skipping: 16, 32, 64 or 128               */
  uint32_t flags;          /* PUREKV_FLAG_DENSE_CAUSAL: plain causal attention;
                              PUREKV_FLAG_COARSE_BLOCKS: widen the mask to whole blocks   */
  int32_t local_window;    /* > 0: also the local_window most recent positions (0: off)    */
  int32_t atrous_dilation; /* > 0: also positions i - D, i - 2D, ... (0: off)              */
} purekv_st_params;

/* Packed batch.  Device arrays feed kernels; host mirrors feed planning and launch sizing.
 * Both must hold the same values. */
typedef struct {
  int32_t n_req;
  int64_t total_tokens;        /* T = h_cu_seqlens[n_req]                                  */
  const int32_t *cu_seqlens;   /* device [n_req+1]                                         */
  const int32_t *h_cu_seqlens; /* host   [n_req+1]                                         */
  const int32_t *h_n_prefix;   /* host   [n_req] text tokens before the video              */
  const int32_t *h_n_frames;   /* host   [n_req]; suffix = len - n_prefix - n_frames*N     */
} purekv_batch;

/* Host-side summary of a built plan; filled by purekv_plan_build, read by
 * purekv_st_sparse_prefill. */
typedef struct {
  int32_t tile_q, tile_k;   /* rows per query tile, keys per key tile                      */
  int32_t n_qtiles;         /* query tiles over all requests                               */
  int32_t max_list;         /* longest kept-tile list of a query tile                      */
  int64_t tiles_kept;       /* key tiles kept (summed over query tiles)                    */
  int64_t tiles_causal;     /* key tiles a dense causal mask would keep                    */
  int64_t pairs_kept;       /* (query, key) pairs the mask keeps                           */
  int64_t tiles_full, tiles_diag, tiles_general; /* kept tiles by predicate class          */
  int64_t bytes_used;       /* bytes of the plan buffer actually written                   */
  int32_t dtype, head_dim;  /* what the plan was built for                                 */
  int32_t n_q_heads, n_kv_heads;
  int32_t n_ctas, n_units;  /* tensor-core kernel: persistent CTAs and their work units    */
  int32_t max_chunks;       /* most chunks a kept-key list was split into                  */
  int64_t ws_bytes;         /* workspace purekv_st_sparse_prefill needs with this plan     */
} purekv_plan_info;

const char *purekv_version(void);
/* Copies the calling thread's last error text (NUL-terminated) into buf. */
void purekv_last_error(char *buf, size_t buf_bytes);

/* Budget rule: w <- min(window, len); k = min(len, max(w, floor(keep_ratio*len))); h = k - w.
 * Host only.  (Sec. 3.1: recent window w plus top-h non-recent keys; budgets are quoted as a
 * fraction of the cache, Tables 1-2.) */
purekv_status purekv_budget(int32_t len, int32_t window, double keep_ratio, int32_t *h_out, int32_t *k_out);

/* ---- planning (host work + one host-to-device copy) --------------------------------- */
/* Size of the plan buffer in bytes for this batch, mask and head layout; 0 on invalid input.
 * n_ctas = number of persistent CTAs the tensor-core kernel is scheduled for (0: 148, one per
 * SM of a B200). */
size_t purekv_plan_bytes(const purekv_batch *batch, const purekv_st_params *params,
                         purekv_dtype dtype, int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads,
                         int32_t n_ctas);
/* Builds, on the host, the per-query-tile lists of key tiles the mask keeps (each tagged
 * full / causal-only / general, the latter with a bit mask), and for the tensor-core kernel
 * its work list: lists longer than about half a CTA's share are split into chunks, and the
 * (query tile, head pair, chunk) units are put in order of decreasing estimated cost; the
 * kernel's n_ctas persistent CTAs draw them in that order as they become free.  The result
 * is copied into `plan` (device, plan_bytes >= purekv_plan_bytes) on `stream`, and the call
 * waits for that copy.  A plan depends only on the batch shape, the mask and the head layout,
 * not on Q/K/V, and serves every layer.  It holds a few counters the kernel uses to hand out
 * units and to combine split lists (they return to zero when a launch ends), so one plan serves one launch at a
 * time: launches that share a plan must be ordered, e.g. on one stream, and a plan whose launch
 * reported PUREKV_ERR_TIMEOUT must be rebuilt. */
purekv_status purekv_plan_build(const purekv_batch *batch, const purekv_st_params *params,
                                purekv_dtype dtype, int32_t head_dim, int32_t n_q_heads,
                                int32_t n_kv_heads, int32_t n_ctas, void *plan, size_t plan_bytes,
                                purekv_plan_info *h_info, void *stream);

/* Same planning, written to a HOST buffer h_plan (plan_bytes >= purekv_plan_bytes); makes no
 * CUDA call.  The bytes may be copied to the device by the caller and used as `plan`. */
purekv_status purekv_plan_build_host(const purekv_batch *batch, const purekv_st_params *params,
                                     purekv_dtype dtype, int32_t head_dim, int32_t n_q_heads,
                                     int32_t n_kv_heads, int32_t n_ctas, void *h_plan,
                                     size_t plan_bytes, purekv_plan_info *h_info);

/* ---- ST-SpAttn prefill, one layer (Sec. 3.2; softmax of Eq. 1 over the kept keys) ------
 * O[i,hq,:] = sum_{j<=i, M(i,j)} softmax_j(scale * q_i.k_j) v_j.   lse (nullable) [H, T] fp32
 * receives log-sum-exp (natural log) of each row's kept logits.  softmax_scale 0 means
 * 1/sqrt(head_dim).  bf16 with head_dim 128 and tile 64/128 runs on the tcgen05 tensor
 * cores; other supported shapes (head_dim 32, 64, 128 or 256) run on CUDA cores.
 * `ws` is a device workspace of at least h_info->ws_bytes bytes (it holds the partial results
 * of split key lists; may be null when ws_bytes is 0); it need not be initialised.
 * `status` (nullable) is a device int32 the kernel sets to PUREKV_ERR_TIMEOUT if a bounded
 * wait expires; the caller zeroes it and reads it (purekv_poll_status). */
purekv_status purekv_st_sparse_prefill(const void *q, const void *k, const void *v, void *o, float *lse,
                                       const purekv_batch *batch, void *plan,
                                       const purekv_plan_info *h_info, int32_t n_q_heads,
                                       int32_t n_kv_heads, int32_t head_dim, purekv_dtype dtype,
                                       float softmax_scale, void *ws, size_t ws_bytes, int32_t *status,
                                       void *stream);

/* ---- low-layer window scores (Eq. 1-2) -------------------------------------------------
 * For request r of length l, w = min(window, l), KV head g, key j < l-w:
 *   C[g, j] = (1/G) sum_{hq in group g} sum_{i=l-w}^{l-1} A^{hq}[i, j],
 * A = dense causal softmax (each row normalised over all keys j' <= i).  c_out [H_kv, T]
 * fp32; the last w entries of each request are written as 0.  The attention matrix is never
 * stored.  ws: device workspace of purekv_score_ws_bytes (log-sum-exp of the window rows and, for the
 * tensor-core path, their per-key-block parts); it need not be initialised. */
size_t purekv_score_ws_bytes(const purekv_batch *batch, int32_t window, int32_t n_q_heads);
purekv_status purekv_lowlayer_score(const void *q, const void *k, float *c_out, const purekv_batch *batch,
                                    int32_t window, int32_t n_q_heads, int32_t n_kv_heads,
                                    int32_t head_dim, purekv_dtype dtype, float softmax_scale,
                                    void *ws, size_t ws_bytes, void *stream);

/* The same scores in one pass, for a layer whose dense causal prefill has already produced the rows' log-sum-exp
 * (Eq. 1's row normaliser): lse is the [H, T] fp32 output of purekv_st_sparse_prefill run on the same Q, K with
 * PUREKV_FLAG_DENSE_CAUSAL (natural log), so C = (1/G) sum over the window rows of exp(s - lse) needs no first
 * pass and no workspace.  Runs on the tcgen05 tensor cores; supports bf16, head_dim 128 and a window that is a
 * multiple of 8 (requests shorter than the window must then have a multiple of 8 tokens), and returns
 * PUREKV_ERR_UNSUPPORTED otherwise -- use purekv_lowlayer_score for those.  `status` as in the prefill call. */
purekv_status purekv_lowlayer_score_lse(const void *q, const void *k, const float *lse, float *c_out,
                                        const purekv_batch *batch, int32_t window, int32_t n_q_heads,
                                        int32_t n_kv_heads, int32_t head_dim, purekv_dtype dtype,
                                        float softmax_scale, int32_t *status, void *stream);

/* ---- the score reductions of other eviction policies (App. A.1, Table 6: the paper drives H2O-, SnapKV- and
 * StreamingLLM-style policies with its estimator and ST-SpAttn; it cites the policies by name, so the forms here are
 * the usual ones of those methods) ------------------------------------------------------------
 * purekv_lowlayer_score_ex is purekv_lowlayer_score with two more parameters:
 *   obs_rows  how many of a request's last rows are accumulated.  obs_rows = window is Eq. 2 itself; a negative
 *             value (or one beyond the request) accumulates every row of A -- the "accumulated attention scores"
 *             of Sec. 3.1, biased toward early keys by the lower-triangular matrix; a small value is the
 *             observation window of SnapKV-style policies.  A row counts only for the keys it can see (j <= i).
 *   pool      odd, >= 1: each non-recent key's sum is replaced by the mean over `pool` positions centred on it,
 *             positions outside the non-recent segment counting as zero (1: no pooling).
 * c_out as in purekv_lowlayer_score (the recent `window` keys get 0), so Eq. 3 / Eq. 4 and the selection apply
 * unchanged.  ws: purekv_score_ex_ws_bytes.  Accumulating all rows costs two passes over the whole causal matrix.
 * purekv_select_sink_recent is the score-free policy (attention sinks + recent window): for every layer and KV
 * head the first h_keep[r] positions of request r, then its window; idx_out as purekv_select_topk writes it. */
size_t purekv_score_ex_ws_bytes(const purekv_batch *batch, int32_t obs_rows, int32_t pool, int32_t n_q_heads,
                                int32_t n_kv_heads);
purekv_status purekv_lowlayer_score_ex(const void *q, const void *k, float *c_out, const purekv_batch *batch,
                                       int32_t window, int32_t obs_rows, int32_t pool, int32_t n_q_heads,
                                       int32_t n_kv_heads, int32_t head_dim, purekv_dtype dtype,
                                       float softmax_scale, void *ws, size_t ws_bytes, void *stream);
purekv_status purekv_select_sink_recent(const purekv_batch *batch, int32_t window, const int32_t *keep /* device */,
                                        const int32_t *h_keep, const int32_t *cu_kept /* device */,
                                        const int32_t *h_cu_kept, int32_t n_layers, int32_t n_kv_heads,
                                        int32_t *idx_out, void *stream);

/* ---- the same scores for callers that cannot hand over a workspace ---------------------------
 * (The paper has no counterpart: this is a packaging variant of purekv_lowlayer_score.)
 * Some callers cannot obtain device memory at the moment they need the scores: a serving engine that
 * gave all of HBM to its KV-cache pool at start-up has nothing left to cudaMalloc from, and code that
 * runs where an allocation would stall the device (cudaMalloc and cudaFree synchronise) must not
 * allocate at all.  For them this entry point keeps its scratch (the window rows' log-sum-exp values)
 * in an array inside the library's device image instead of a caller-provided workspace.  It calls no
 * cudaMalloc / cudaFree and no allocating library routine; inputs and c_out are still the caller's.
 *  - Limit: the problem's workspace need in fp32 values -- with rows = n_req * n_q_heads * max(window, 1):
 *    rows rounded up to a multiple of 64, plus 2 * rows * ceil(longest request / 64) -- must not exceed
 *    PUREKV_NOALLOC_SCORE_MAX_ROWS (262144) values: 1 MiB that every GPU loading the library holds until the
 *    process exits (a 2432-token prompt with 32 query heads and a window of 64 needs 157 696).  Larger problems
 *    return PUREKV_ERR_WORKSPACE and leave c_out untouched; use purekv_lowlayer_score.  An empty batch returns
 *    PUREKV_OK whatever the other arguments are.
 *  - The first call on each device looks up the array's device address (with that device current).
 *    Make that first call before any stream capture on that device.
 *  - All calls on a device share the one array, and it keeps the previous call's contents.  Nothing in
 *    it has to start at zero (each call overwrites every entry it later reads), but two calls whose
 *    kernels overlap on the GPU -- different streams, or different host threads -- race on it.
 *    Serialise them, e.g. by issuing them on one stream.
 * Results are those of purekv_lowlayer_score. */
#define PUREKV_NOALLOC_SCORE_MAX_ROWS 262144
purekv_status purekv_lowlayer_score_noalloc(const void *q, const void *k, float *c_out,
                                            const purekv_batch *batch, int32_t window, int32_t n_q_heads,
                                            int32_t n_kv_heads, int32_t head_dim, purekv_dtype dtype,
                                            float softmax_scale, void *stream);

/* ---- V-norm weighting and top-h selection, n_layers layers per call (Eq. 3-4) ----------
 * S[L, g, j] = C[g, j] * ||V_L[j, g, :]||_2 for non-recent j; idx[L, g, cu_kept[r] + t] lists,
 * for request r, the h_keep[r] positions with the largest S (ties: lower position), in
 * ascending position order, followed by the window positions l-w .. l-1.  Positions are
 * relative to the request.  v is [n_layers][T, H_kv, d] with v_layer_stride elements between
 * layers.  idx_out [n_layers, H_kv, K_tot] int32, K_tot = h_cu_kept[n_req];
 * cu_kept[r+1]-cu_kept[r] must equal h_keep[r] + min(window, l_r).
 * s_out (nullable) [n_layers, H_kv, T] fp32 receives S.  ws: purekv_select_ws_bytes. */
size_t purekv_select_ws_bytes(const purekv_batch *batch, int32_t n_layers, int32_t n_kv_heads);
purekv_status purekv_select_topk(const float *c, const void *v, int64_t v_layer_stride, int32_t n_layers,
                                 const purekv_batch *batch, int32_t window, const int32_t *keep /* device [n_req] */,
                                 const int32_t *h_keep, const int32_t *cu_kept /* device [n_req+1] */,
                                 const int32_t *h_cu_kept, int32_t n_kv_heads, int32_t head_dim,
                                 purekv_dtype dtype, int32_t *idx_out, float *s_out, void *ws,
                                 size_t ws_bytes, void *stream);

/* ---- selection and compaction in one call (Sec. 3.1: the selection feeds the compressed cache directly) ----
 * purekv_select_topk followed by purekv_compact_kv of the same layers, in the selection's own kernels: the CTA
 * that has chosen a (request, KV head, layer) segment's positions copies those K and V rows (k and v share
 * layer_stride) into k_out / v_out [n_layers][K_tot, H_kv, d] (out_layer_stride) -- one launch fewer, and the
 * indices do not travel through memory between two kernels.  idx_out (and s_out, if given) are written as by
 * purekv_select_topk; results are bit-identical to the two separate calls. */
purekv_status purekv_select_compact(const float *c, const void *k, const void *v, int64_t layer_stride,
                                    int32_t n_layers, const purekv_batch *batch, int32_t window,
                                    const int32_t *keep /* device [n_req] */, const int32_t *h_keep,
                                    const int32_t *cu_kept /* device [n_req+1] */, const int32_t *h_cu_kept,
                                    int32_t n_kv_heads, int32_t head_dim, purekv_dtype dtype, int32_t *idx_out,
                                    float *s_out, void *k_out, void *v_out, int64_t out_layer_stride, void *ws,
                                    size_t ws_bytes, void *stream);

/* ---- compaction (the compressed cache of Sec. 3.1) -------------------------------------
 * k_out[L, cu_kept[r]+t, g, :] = k[L, cu_seqlens[r] + idx[L, g, cu_kept[r]+t], g, :], same for v.
 * k, v: [n_layers][T, H_kv, d] with layer_stride elements between layers; outputs
 * [n_layers][K_tot, H_kv, d] with out_layer_stride.  Pure copy, 128-bit vectorised; d * element
 * size must be a multiple of 16 bytes and all bases 16-byte aligned. */
purekv_status purekv_compact_kv(const void *k, const void *v, int64_t layer_stride, int32_t n_layers,
                                const int32_t *idx, const purekv_batch *batch, const int32_t *cu_kept,
                                const int32_t *h_cu_kept, int32_t n_kv_heads, int32_t head_dim,
                                purekv_dtype dtype, void *k_out, void *v_out, int64_t out_layer_stride,
                                void *stream);

/* ---- decode step over the compacted cache, one layer per call (Sec. 3.1; the stage Table 3
 * times as decode latency) ---------------------------------------------------------------
 * o[r, hq, :] = sum_j softmax_j(q[r, hq, :] . k_cache[j, hq / G, :] * scale) * v_cache[j, hq / G, :]
 * over the kept rows j = cu_kept[r] .. cu_kept[r+1]-1 of request r: one new query per request
 * and head, every kept key visible.  q, o: [n_req, H, d] (dtype); k_cache, v_cache:
 * [K_tot, H_kv, d] as written by purekv_compact_kv for one layer; lse (nullable): [n_req, H]
 * fp32, natural log.  A request with no kept row gets o = 0 and lse = -inf.  Rows must be 256
 * bytes (bf16 with d = 128, fp32 with d = 64) and G = H / H_kv at most 16 (bf16) or 8 (fp32),
 * else PUREKV_ERR_UNSUPPORTED.  All device pointers 16-byte aligned; cu_kept on the device and
 * h_cu_kept on the host hold the same n_req + 1 offsets.  ws: purekv_decode_ws_bytes for the
 * largest per-request count (may be NULL when that returns 0); nothing is allocated, nothing
 * synchronises.  softmax_scale <= 0 means 1/sqrt(d). */
size_t purekv_decode_ws_bytes(int32_t n_req, int32_t max_kept, int32_t n_q_heads, int32_t n_kv_heads,
                              int32_t head_dim);
purekv_status purekv_decode_attention(const void *q, const void *k_cache, const void *v_cache, void *o,
                                      float *lse, const int32_t *cu_kept /* device [n_req+1] */,
                                      const int32_t *h_cu_kept, int32_t n_req, int32_t n_q_heads,
                                      int32_t n_kv_heads, int32_t head_dim, purekv_dtype dtype,
                                      float softmax_scale, void *ws, size_t ws_bytes, void *stream);

/* Failure detection (no counterpart in the paper).  Every wait inside the tensor-core kernels -- on a copy, on a
 * product, on another role of the CTA -- is bounded: when the limit passes the CTA raises the status word to
 * PUREKV_ERR_TIMEOUT, lets its copies and products in flight finish, frees its tensor memory and returns, so the
 * context stays usable.  The limit is process-wide, 1 s by default; ns == 0 restores the default.  The tensor-core
 * prefill also checks the plan before using it (header, section offsets against the plan's size, every unit's and
 * entry's indices against the header's counts): on a mismatch nothing is read through the bad field, the status
 * word becomes PUREKV_ERR_BAD_PLAN and the output is undefined (untouched when the header itself fails).  After either code the plan's scheduling counters are
 * undefined: build the plan again before the next launch. */
void purekv_set_wait_limit_ns(uint64_t ns);

/* Synchronises `stream`, copies the device status word to *h_status_out and returns the code it holds
 * (PUREKV_ERR_TIMEOUT or PUREKV_ERR_BAD_PLAN) if it is non-zero, PUREKV_ERR_CUDA if the stream reported an error.
 * status == NULL polls the word inside the library that calls made with a NULL status use (one per
 * device, shared by all such calls) and clears it if it was raised.  A raised word makes every later
 * call that uses it return without computing -- the caller's own word stays raised until the caller
 * clears it, the library's until it is polled this way -- so poll after the calls whose results matter. */
purekv_status purekv_poll_status(const int32_t *status, int32_t *h_status_out, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* PUREKV_H_ */
