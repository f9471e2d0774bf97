/*
 * hkv.h — C ABI of the HybridKV decode hot path for NVIDIA B200 (sm_100a).
 *
 * One autoregressive step of attention over a hybrid-compressed KV cache, and the compression that
 * builds that cache (paper: Section 3.3 "Hybrid KV Cache Compression" and Appendix A "Details of
 * Hybrid KV Cache Compression").
 *
 *   static  KV heads: text-prior static pruning — the cache keeps (i) the observation window,
 *                     (ii) every text token before it, (iii) the Top-M visual tokens before it by
 *                     the window score s_w; decode attends densely over that compacted cache.
 *   dynamic KV heads: chunk-wise retrieval — the sequence is cut into fixed-size chunks, each
 *                     represented by the mean of its keys; every decode step scores the query
 *                     against the chunk means, takes the top-k chunks its budget allows and attends
 *                     over the tokens of those chunks only.
 *
 * "Head" always means KV head; the G = n_q_heads / n_kv_heads query heads of a group share it.
 *
 * Conventions
 *   - plain C linkage; no exception crosses the boundary; every call returns a status.  Argument
 *     errors are found on the host before anything is launched.  Global state is limited to a
 *     helper stream with a few events per device (hkv_compress builds the dynamic heads on it beside
 *     the static ones, hkv_decode_step_host runs its copies on it; both fork it from and join it to
 *     the caller's stream, so the caller sees one ordered stream) and the fixed scratch of
 *     hkv_topk_chunks_noalloc.  hkv_compress uploads its plan from ordinary host memory that it frees
 *     on return, so it is not a call to capture in a CUDA graph; the decode calls are.
 *   - "dev" pointers are device (HBM) addresses on the current CUDA device, "host" pointers are
 *     ordinary host memory.  bf16 tensors are passed as void*.
 *   - the caller owns every device buffer, including cache_mem and workspace.  The library never
 *     allocates or frees device memory.  The opaque handle owns host metadata only.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  All device
 *     work is enqueued on it; calls return without synchronising unless stated.
 *   - dense tensors are row-major with the last index fastest.
 */
#ifndef HKV_H_
#define HKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  HKV_OK = 0,
  HKV_ERR_INVALID_ARG = 1, /* NULL pointer, negative size, bad index                         */
  HKV_ERR_SHAPE = 2,       /* inconsistent geometry (lengths, window, heads)                   */
  HKV_ERR_BUDGET = 3,      /* a budget < 1                                                     */
  HKV_ERR_WORKSPACE = 4,   /* cache_mem / workspace too small or misaligned (256 B)            */
  HKV_ERR_UNSUPPORTED = 5, /* geometry outside what the kernels are built for                  */
  HKV_ERR_CUDA = 6,        /* a CUDA runtime call failed                                       */
  HKV_ERR_TIMEOUT = 7,     /* a bounded device-side wait ran out (see hkv_last_device_error)   */
  HKV_ERR_INDEX = 8        /* a device-side index check failed                                 */
} hkv_status;

/* flags */
#define HKV_CAUSAL_WINDOW 1u /* mask key j > position of the window row inside S_w (variant; the
                                paper's equation has no mask)                                  */
#define HKV_OUT_F32 2u       /* hkv_decode_attn writes float32 instead of bf16                 */
#define HKV_GROUP_MAX 4u     /* chunk score of a GQA group = the largest of its query heads' inner
                                products with the chunk mean instead of their sum (variant: the
                                paper scores per head and does not say how a shared KV head
                                combines its group)                                            */

#define HKV_OFFLOAD_DYNAMIC 8u /* the K/V planes of the dynamic heads live in pinned host memory and
                                the selected chunks cross PCIe every step (the paper's own
                                placement, Section 3.3 / Appendix A); only with hkv_plan_offload /
                                hkv_compress_offload                                           */

/* Geometry of one layer's cache.  Supported: head_dim = 128, 1 <= n_q_heads / n_kv_heads <= 16,
 * chunk_size >= 1, 1 <= obs_window <= every seq_len. */
typedef struct {
  int32_t batch;         /* B                                                                  */
  int32_t n_q_heads;     /* Hq                                                                 */
  int32_t n_kv_heads;    /* Hkv                                                                */
  int32_t head_dim;      /* d                                                                  */
  int32_t max_seq_len;   /* C_max: row pitch of k, v, is_text, token_scores                    */
  int32_t chunk_size;    /* cs: tokens per chunk of a dynamic head (Appendix A)                */
  int32_t obs_window;    /* w: length of the observation window (Appendix A)                   */
  float softmax_scale;   /* 0 -> 1/sqrt(head_dim); used by S_w and by decode attention         */
  uint32_t flags;
  int32_t append_capacity; /* tokens hkv_append may add to every sequence after compression (0 = none) */
} hkv_config;

typedef struct hkv_cache hkv_cache; /* opaque; host metadata of one layer's compressed cache */

typedef struct {
  int64_t retained_tokens;       /* sum over heads of tokens attended per step (upper bound for
                                    dynamic heads: k * cs)                                     */
  int64_t kv_bytes_resident;     /* bytes of K/V planes held in cache_mem                      */
  int64_t summary_bytes;         /* bytes of chunk means held in cache_mem                     */
  int64_t algorithmic_bytes_per_step; /* 512 B per retained token + 256 B per chunk mean read  */
  int64_t cache_bytes;           /* bytes of cache_mem in use                                  */
  int64_t workspace_bytes;       /* bytes of compress workspace required                       */
  int32_t n_static, n_dynamic;   /* (b, h) units of each type                                  */
  int32_t n_splits;              /* CTAs of a decode launch on this cache alone (units x cluster size) */
  int32_t launches_per_decode;   /* kernels one hkv_decode_attn enqueues (1: score, select, attend and
                                    merge are one kernel)                                      */
} hkv_stats;

/* Sizes of the two caller-owned device buffers, from HOST inputs only (no device work, no sync).
 * The keep-set of a static head always has min(budget, seq_len) tokens and a dynamic head always
 * loads min(n_chunks, ceil(budget / cs)) chunks (Appendix A, second paragraph: the number of chunks
 * follows from the head's budget and the chunk size), so no size depends on device data.
 *   seq_lens  host int32 [B]        token count C_b of each sequence, 1 <= C_b <= max_seq_len
 *   head_type host uint8 [B, Hkv]   0 = static, 1 = dynamic (Section 3.1's classification result)
 *   budgets   host int32 [B, Hkv]   per-head token budget (Section 3.2's allocation result), >= 1;
 *                                   values above C_b are clamped to C_b
 * Out: bytes for cache_mem (lives as long as the cache) and for workspace (needed only until the
 * work hkv_compress enqueued has finished). */
hkv_status hkv_plan(const hkv_config* cfg, const int32_t* seq_lens, const uint8_t* head_type,
                    const int32_t* budgets, size_t* cache_bytes, size_t* workspace_bytes);

/* Build one layer's compressed cache (Appendix A, both paragraphs).
 *   k, v         dev bf16 [B, Hkv, C_max, d]   full prefill keys / values (read only)
 *   q_obs        dev bf16 [B, w, Hq, d]        queries of the last w prompt tokens of each sequence
 *                                              (Q[C-w:C] of Appendix A's S_w); may be NULL iff
 *                                              token_scores is given
 *   token_scores dev f32  [B, Hkv, C_max]      optional: replaces s_w for static heads
 *   is_text      dev u8   [B, C_max]           1 = text token, 0 = visual token
 *   seq_lens, head_type, budgets               host arrays as in hkv_plan
 *   cache_mem    dev, >= cache_bytes, 256-B aligned; owned by the caller, must outlive the handle's
 *                use; holds the compacted static K/V, the dynamic K/V and chunk means, index lists
 *                and the decode scratch
 *   workspace    dev, >= workspace_bytes, 256-B aligned; may be released once the stream has
 *                passed the work of this call
 * Static head: s_w = mean over the w*G window rows of softmax(q k^T * scale) over all C_b tokens;
 * keep = window U text-before-window U Top-M visual-before-window (M = budget - w - #text), ties to
 * the lower position; if the budget cannot hold window + text, text is ranked by s_w for the
 * budget - w places left; if budget <= w the last `budget` tokens are kept.
 * Dynamic head: chunk mean = float32 sum of the chunk's keys in token order / chunk length, rounded
 * to nearest-even bf16; the last chunk may be shorter.
 * k, v, q_obs, token_scores and is_text may be released once the stream has passed this call.
 * The window-score kernels (and hkv_classify_heads) run on the tcgen05 tensor cores: while they run,
 * each of their thread blocks holds all tensor memory and nearly all shared memory of its SM, so
 * kernels of other streams that need tensor memory wait for them.
 * On success *out receives a handle to free with hkv_cache_destroy. */
hkv_status hkv_compress(const hkv_config* cfg, const void* k, const void* v, const void* q_obs,
                        const float* token_scores, const uint8_t* is_text, const int32_t* seq_lens,
                        const uint8_t* head_type, const int32_t* budgets, void* cache_mem,
                        size_t cache_bytes, void* workspace, size_t workspace_bytes, void* stream,
                        hkv_cache** out);

/* The paper's placement of the dynamic heads' KV (Section 3.3: dynamic-head KV is offloaded to CPU
 * memory and the chunks a step selects are fetched to the GPU; Appendix A).  Same as hkv_plan /
 * hkv_compress with cfg->flags carrying HKV_OFFLOAD_DYNAMIC, except that the K and V planes of the
 * dynamic heads are written to `host_mem` instead of cache_mem (chunk means, scores and index lists
 * stay on the device).
 *   host_mem   pinned host memory the device can address at the same pointer value (cudaHostAlloc /
 *              cudaMallocHost / a registered range under unified addressing), >= host_bytes, 256-B
 *              aligned, owned by the caller, alive as long as the handle is used
 * Every later call on the handle (decode, append, getters) works unchanged: the decode kernel's bulk
 * copies read the selected chunks straight from host memory, so a step moves them over PCIe and no
 * staging buffer or extra launch exists.  Without dynamic heads host_bytes is 0 and host_mem may be
 * NULL.  The plain hkv_plan / hkv_compress reject the flag (HKV_ERR_INVALID_ARG), and these two
 * reject its absence. */
hkv_status hkv_plan_offload(const hkv_config* cfg, const int32_t* seq_lens, const uint8_t* head_type,
                            const int32_t* budgets, size_t* cache_bytes, size_t* workspace_bytes,
                            size_t* host_bytes);
hkv_status hkv_compress_offload(const hkv_config* cfg, const void* k, const void* v, const void* q_obs,
                                const float* token_scores, const uint8_t* is_text, const int32_t* seq_lens,
                                const uint8_t* head_type, const int32_t* budgets, void* cache_mem,
                                size_t cache_bytes, void* host_mem, size_t host_bytes, void* workspace,
                                size_t workspace_bytes, void* stream, hkv_cache** out);

/* One decode step over the compressed cache (Appendix A: score chunks by the inner product of the
 * query with the chunk metadata, take the top chunks, attend together with the static cache).
 *   q    dev bf16 [B, Hq, d]   the step's query
 *   out  dev bf16 [B, Hq, d]   (float32 if HKV_OUT_F32) attention output
 * Dynamic head: score_c = sum over the group's query heads of <q_g, mean_c> (float32), top-k with
 * ties to the lower chunk id, softmax attention over the tokens of the selected chunks.  Static
 * head: softmax attention over its kept tokens.  Heads are independent.  Allocates nothing, never
 * synchronises, results are deterministic.  q must be 4-byte and out 16-byte aligned.  Calls on the
 * same cache must not overlap on the GPU (they share the cache's scratch).  One kernel launch; when
 * it follows another decode launch on the stream it is launched with programmatic stream
 * serialisation: it may start early, but reads q and writes anything only once everything enqueued
 * before it has completed. */
hkv_status hkv_decode_attn(hkv_cache* cache, const void* q, void* out, void* stream);

/* Decode several layers' caches with ONE launch sequence: queries q[i] / outputs out[i] belong to
 * caches[i].  All caches must have been planned with the same geometry.  Benchmark aid for small
 * per-layer work; a real model's layers are sequential.  host arrays of n pointers. */
hkv_status hkv_decode_attn_multi(hkv_cache* const* caches, const void* const* q, void* const* out,
                                 int32_t n, void* stream);

/* The two stages of hkv_decode_attn as separate calls (hkv_decode_attn = hkv_select_chunks followed
 * by hkv_attend on the same stream).  hkv_select_chunks scores every chunk of every dynamic head
 * against q and stores the top-k chunk ids in the cache (Appendix A, second paragraph: chunk relevance
 * is the query's inner product with the chunk metadata).  hkv_attend runs the attention of all heads
 * over the static cache and the currently stored selection (same paragraph: the output is computed
 * over the static cache and the loaded chunks together); it needs one earlier hkv_select_chunks (or
 * hkv_decode_attn) if the cache has dynamic heads.  Same pointer rules. */
hkv_status hkv_select_chunks(hkv_cache* cache, const void* q, void* stream);
hkv_status hkv_attend(hkv_cache* cache, const void* q, void* out, void* stream);

/* hkv_decode_attn with HOST buffers: copies q_host -> q_dev, runs the step, copies out_dev ->
 * out_host, all enqueued on `stream` (the result is in out_host once the stream has passed the call).
 *   q_host, out_host  host memory (pinned for truly asynchronous copies), shapes as q / out
 *   q_dev, out_dev    caller-owned device staging buffers of the same sizes */
hkv_status hkv_decode_attn_host(hkv_cache* cache, const void* q_host, void* out_host, void* q_dev,
                                void* out_dev, void* stream);

/* Adds the token just generated to the compressed cache of one layer (Appendix A and Section 3.3 only
 * say that the GPU KV buffer keeps changing while decoding proceeds).  Reading taken here, the paper
 * giving no rule: the new token's key / value row of
 *   a static head   is appended to its condensed cache and is always retained (it is the most
 *                   recent context);
 *   a dynamic head  joins the chunked sequence: it goes to the open last chunk (or opens a new one),
 *                   whose metadata is recomputed as the float32 running sum of its keys in token
 *                   order / its length, rounded to bf16 — bit-identical to building the metadata
 *                   of the longer sequence from scratch; the number of chunks loaded per step
 *                   follows the unchanged budget.
 *   k_new, v_new  dev bf16 [B, Hkv, d]   the new token's key and value of every KV head
 * Every sequence grows by one token per call, at most hkv_config.append_capacity times
 * (HKV_ERR_WORKSPACE afterwards).  Enqueued on `stream`, no synchronisation; must not overlap a
 * decode call on the same cache. */
hkv_status hkv_append(hkv_cache* cache, const void* k_new, const void* v_new, void* stream);

/* One decode step of a whole model with HOST buffers (Appendix A's per-step procedure, layer after
 * layer): the queries of the first layer are copied to the device on `stream`, those of the other
 * layers meanwhile on a second stream the library keeps per device; one hkv_decode_attn launch per
 * layer follows on `stream` (caches[i] with layer i's slice, in order); the outputs return in four
 * groups of layers, the first three beside the layers still running, the last on `stream`, which
 * also waits for the second stream before the call's work counts as finished.  From the caller's
 * side everything is ordered on `stream`; the call may be captured in a CUDA graph (the second
 * stream forks from and joins `stream` by events).  The first call on a device creates that stream
 * and its events.
 *   q_host, out_host  host [n, B, Hq, d] (pinned for truly asynchronous copies); bf16 / float32 as for hkv_decode_attn
 *   q_dev, out_dev    caller-owned device staging buffers of the same sizes
 * All caches must share one geometry (batch, heads, output type). */
hkv_status hkv_decode_step_host(hkv_cache* const* caches, int32_t n, const void* q_host, void* out_host,
                                void* q_dev, void* out_dev, void* stream);

hkv_status hkv_cache_destroy(hkv_cache* cache);

/* Top-down budget allocation (Section 3.2, both paragraphs): from a total token budget to the
 * per-head budgets hkv_plan / hkv_compress take.  Host arithmetic in double precision, no device.
 *   n_heads      heads the total is shared by (all layers' KV heads of one sequence, in any fixed order)
 *   head_type    host u8 [n_heads]   0 = static, 1 = dynamic (Section 3.1)
 *   scores       host f64 [n_heads]  text-centric sparsity score S_{l,h} >= 0 of each head (only static
 *                                    heads' entries are read); NULL = all equal
 *   total_budget B_total in tokens, >= n_heads
 *   r            share coefficient of the dynamic heads, 0 < r <= B_total / (B_bar * N_dyna)
 *   alpha        in [0, 1]: weight of the uniform base budget against the score-proportional one
 *   flags        HKV_BUDGET_PAD_POW2: round the dynamic per-head budget up to a power of two
 *   budgets_out  host int32 [n_heads]
 * Head-type level:  B_bar = B_total / (N_stat + N_dyna);  B_dyna = ceil(r * B_bar * N_dyna);
 * B_stat = B_total - B_dyna.  Static head:  b = ceil(alpha * B_stat / N_stat + (1 - alpha) * B_stat * S~),
 * S~ = S / sum of S over all static heads.  Dynamic head:  ceil(B_dyna / N_dyna), the same for all.
 * Errors: HKV_ERR_BUDGET if r breaks its bound, if the total cannot give every head one token, or
 * alpha is outside [0, 1]. */
#define HKV_BUDGET_PAD_POW2 1u
hkv_status hkv_allocate_budgets(int32_t n_heads, const uint8_t* head_type, const double* scores,
                                int64_t total_budget, double r, double alpha, uint32_t flags,
                                int32_t* budgets_out);

/* Text-centric head classification (Section 3.1, with the text-centric attention of Section 2.1):
 * for every (sequence b, kv head h), S_text = softmax(Q_text K^T * scale) row by row over ALL C_b
 * context tokens (no mask), the sum of each row's k_b = max(1, ceil(topk_fraction * C_b)) largest
 * entries, and their mean over the rows: the text-centric sparsity score S in (0, 1].  A head is
 * static (0) if S >= theta, else dynamic (1).  Under grouped-query attention the rows of a kv head
 * are the text positions of every query head of its group (n_text[b] * G rows).
 *   cfg          batch, n_q_heads, n_kv_heads, head_dim (128), max_seq_len, softmax_scale are read
 *   k            dev bf16 [B, Hkv, max_seq_len, d]  keys of the prompt, as for hkv_compress
 *   q_text       dev bf16 [B, n_text_max, Hq, d]    queries of the text tokens; rows >= n_text[b] are not read
 *   seq_lens     host int32 [B]  C_b in 1..max_seq_len;   n_text  host int32 [B]  in 1..n_text_max
 *   topk_fraction in (0, 1] (the paper's focus fraction is 0.05);  theta finite (the paper settles on 0.9)
 *   workspace    dev, 256-B aligned, >= min_bytes of hkv_classify_workspace; with less than
 *                preferred_bytes the rows are processed in several passes (same result)
 *   scores_out   dev f64 [B, Hkv]  S (float32 softmax arithmetic, rows averaged in double, fixed order)
 *   head_type_out dev u8 [B, Hkv]  the array hkv_plan / hkv_compress take, once copied to the host
 * Enqueued on `stream`, no synchronisation; deterministic.  Errors: HKV_ERR_SHAPE (lengths),
 * HKV_ERR_WORKSPACE, HKV_ERR_UNSUPPORTED (head_dim), HKV_ERR_INVALID_ARG. */
hkv_status hkv_classify_workspace(const hkv_config* cfg, int32_t n_text_max, size_t* min_bytes,
                                  size_t* preferred_bytes);
hkv_status hkv_classify_heads(const hkv_config* cfg, const void* k, const void* q_text, int32_t n_text_max,
                              const int32_t* seq_lens, const int32_t* n_text, double topk_fraction,
                              double theta, void* workspace, size_t workspace_bytes, double* scores_out,
                              uint8_t* head_type_out, void* stream);

/* Chunk scoring + top-k for one dynamic head WITHOUT any caller- or library-allocated scratch.
 * (The paper has no counterpart: this is a packaging variant of the selection step of
 * hkv_select_chunks.)  It exists for callers that cannot allocate device memory where they call
 * from — code running inside another runtime's callback or a latency-critical loop, where
 * cudaMalloc (or a framework allocator) is forbidden or would synchronise the device.  They pass
 * inputs and the output only; the float32 score per chunk, which the other entry points keep in
 * cache_mem, lives in a fixed array inside the library (HKV_NOALLOC_MAX_CHUNKS floats = 256 KiB,
 * held by every GPU that loads the library until the process exits).
 *   q        dev bf16 [group, 128]      the query heads that share the KV head
 *   means    dev bf16 [n_chunks, 128]   chunk means, plain row-major (16-byte aligned)
 *   group    1..16;  n_chunks 1..HKV_NOALLOC_MAX_CHUNKS (more -> HKV_ERR_WORKSPACE);  k >= 1
 *   out_ids  dev int32 [min(k, n_chunks)]  ids of the k highest-scoring chunks, ascending; score =
 *            sum over the group of <q_g, mean_c> in float32, ties to the lower id
 * Allocates nothing and never synchronises.  The first call on each device looks up the array's
 * device address (current device = the one that will run the call); make that first call outside
 * any stream capture.  All calls on a device share the one array and it keeps the last call's
 * scores (every entry in use is rewritten before it is read, nothing needs clearing): two calls
 * that overlap on the GPU, on any streams, race — serialise them. */
#define HKV_NOALLOC_MAX_CHUNKS 65536
hkv_status hkv_topk_chunks_noalloc(const void* q, const void* means, int32_t group, int32_t n_chunks,
                                   int32_t k, int32_t* out_ids, void* stream);

/* ---- introspection (parity tests, roofline numerator). These synchronise the given stream. ---- */

/* kept positions of static head (b, h), ascending; host_out has room for `capacity` ints. */
hkv_status hkv_get_static_indices(hkv_cache* cache, int32_t b, int32_t h, int32_t* host_out,
                                  int32_t capacity, int32_t* n, void* stream);
/* chunk ids the last hkv_decode_attn selected for dynamic head (b, h), ascending. */
hkv_status hkv_get_selected_chunks(hkv_cache* cache, int32_t b, int32_t h, int32_t* host_out,
                                   int32_t capacity, int32_t* n, void* stream);
/* float32 chunk scores of the last hkv_decode_attn for dynamic head (b, h); n = n_chunks. */
hkv_status hkv_get_chunk_scores(hkv_cache* cache, int32_t b, int32_t h, float* host_out,
                                int32_t capacity, int32_t* n, void* stream);
/* bf16 chunk means of dynamic head (b, h), [n_chunks, d] as uint16 bit patterns. */
hkv_status hkv_get_summaries(hkv_cache* cache, int32_t b, int32_t h, uint16_t* host_out,
                             int32_t capacity_rows, int32_t* n_chunks, void* stream);
/* byte offset inside `workspace` of the float32 s_w [C_b] that hkv_compress computed for static
 * head (b, h) (valid while the caller keeps the workspace). */
hkv_status hkv_window_scores_offset(const hkv_cache* cache, int32_t b, int32_t h, size_t* offset);

hkv_status hkv_cache_stats(const hkv_cache* cache, hkv_stats* stats);

/* How many thread-block clusters of 1, 2, ..., 16 CTAs of the decode kernel (for a group of `group`
 * query heads per KV head) the current device can hold at once: max_active_clusters[c - 1] for size
 * c, 16 entries.  hkv_decode_attn picks, per launch, the largest even cluster size (or 1) whose
 * capacity covers all (sequence, KV head) units of the launch and that leaves every CTA at least
 * two tiles, but no more than ten CTAs per unit when the token lists are short (Appendix A's
 * per-head work is what a cluster owns).  Needs a device. */
hkv_status hkv_decode_cluster_capacity(int32_t group, int32_t* max_active_clusters);

/* Device error word: code is HKV_OK, HKV_ERR_TIMEOUT or HKV_ERR_INDEX; detail identifies the place.
 * Synchronises the stream. */
hkv_status hkv_last_device_error(hkv_cache* cache, int32_t* code, int32_t* detail, void* stream);

const char* hkv_status_string(hkv_status s);

/* ---- development builds only: these symbols are NOT in libhkv.so ----
 * Two further builds of the same sources exist beside the product library (build.py: build_checked,
 * build_profile).  Neither changes what any call above computes. */
#ifdef HKV_CHECKED
/* Checked build (-DHKV_CHECKED, with a wait limit of a fraction of a second): the decode kernel
 * validates every index that feeds an address (HKV_ERR_INDEX, the access is skipped).  This call
 * launches one thread block that waits, bounded, on a barrier nothing ever arrives on: it must return
 * by itself and leave HKV_ERR_TIMEOUT / detail 6 in the cache's error word, exactly as a lost copy
 * would inside a decode step (Appendix A's per-step chunk load is where that could happen). */
hkv_status hkv_selftest_wait_timeout(hkv_cache* cache, void* stream);
/* Checked build: puts the cache's error word back to (0, 0); enqueued on `stream`. */
hkv_status hkv_clear_device_error(hkv_cache* cache, void* stream);
#endif
#ifdef HKV_PROFILE
/* Profiling build (-DHKV_PROFILE): thread 0 of every decode CTA writes the global nanosecond timer at
 * the phase boundaries of the kernel (32 slots of 8 bytes per CTA) into `dev_buffer`, successive
 * launches taking successive regions; launches that no longer fit are not recorded.  NULL detaches. */
int hkv_profile_attach(void* dev_buffer, long long n_ctas);
#endif

#ifdef __cplusplus
}
#endif
#endif /* HKV_H_ */
