/*
 * corm.h — C ABI of the CORM hot path for NVIDIA B200 (sm_100a).
 *
 * CORM ("Cache Optimization with Recent Message") evicts a cached key/value pair once the key has been judged
 * minor by every one of the last w queries (Definition 4.1 with the window of the "Approach" paragraph), where a
 * key is important for the query of step t iff its softmax probability is at least alpha/t (Definition 3.1; the
 * paper uses alpha = 1), and never evicts the r most recent tokens (Algorithm 1). The policy runs per head and per
 * layer; with grouped-query attention a shared KV head keeps a key while any query head of its group still needs
 * it (Section 5, "Integrate into grouped-query attention").
 *
 * A "unit" is one (layer, sequence, kv head). Each unit owns a slab of max_tokens slots holding K rows, V rows,
 * one 32-bit verdict register per key and the key's absolute 1-based token position (in a paged cache,
 * corm_cache_create_paged, the K and V rows of a slot live in 32-key pages drawn from a pool the layer's units share;
 * slots, their order and everything below are the same). Register encodings: for
 * window_w <= 32 a shift register (bit b = verdict of the query b steps ago); for 33..256 (the paper's experiments
 * use up to 256) the absolute step of the latest query that found the key important, 0 if none has, which decides
 * Algorithm 1's any() over the last w rows as step_now - register < w. Live entries occupy slots [0, live_len); their slot ORDER IS NOT the token order once decode
 * steps have evicted keys (holes are filled from the tail), so recency is always decided from the stored position.
 *
 * Conventions
 *  - Every pointer argument says "device" or "host". Device buffers are owned by the caller, including the
 *    arena; the library never allocates or frees device memory. corm_cache_t owns host metadata only.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream). Calls that enqueue work are
 *    asynchronous; all calls on one cache must be issued in stream order (they share scratch inside the arena).
 *  - Tensors are row-major and dense; kv_dtype is the element type of the cache, q, k_new, v_new and out.
 *  - Host-detectable errors return a status and enqueue nothing. Device-detected ones (a unit that would exceed
 *    max_tokens) set a sticky device status, skip that unit, never trap or hang, and show in corm_cache_stats.
 */
#ifndef CORM_H_
#define CORM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct corm_cache corm_cache_t;

typedef enum {
    CORM_OK = 0,
    CORM_ERR_INVALID_ARG = 1,
    CORM_ERR_UNSUPPORTED = 2,
    CORM_ERR_ARENA_TOO_SMALL = 3,
    CORM_ERR_STATE = 4,
    CORM_ERR_CUDA = 5,
    CORM_ERR_CAPACITY = 6,
    CORM_ERR_TIMEOUT = 7,
    CORM_ERR_INTERNAL = 8    /* a kernel met an index outside its range (a broken page table, a misplaced buffer):
                                the access was skipped; the cache must be reset */
} corm_status_t;

typedef enum { CORM_F32 = 0, CORM_BF16 = 1 } corm_dtype_t;

typedef struct {
    int32_t n_layers, batch, n_q_heads, n_kv_heads; /* n_q_heads % n_kv_heads == 0, group size in {1,2,4,8} */
    int32_t head_dim;                                /* 64 or 128 */
    int32_t max_tokens;                              /* slab capacity per unit: >= longest prompt + decode steps;
                                                        at most 524288 (UNSUPPORTED beyond) */
    int32_t window_w;                                /* 1..256 recent queries; see the register encodings below */
    int32_t recent_r;                                /* >= 1 (Algorithm 1's slice of the last r entries) */
    float   alpha;                                   /* >= 0; threshold alpha/t; 0 means nothing is ever evicted */
    int32_t kv_dtype;                                /* corm_dtype_t */
    int32_t device;                                  /* CUDA device ordinal of the arena */
} corm_config_t;

typedef struct {
    int64_t live_keys, appended_keys, evicted_keys; /* summed over all units */
    double  retention;                               /* live / appended (1 when nothing was appended) */
    int64_t kv_bytes_live, aux_bytes_live;           /* K+V bytes; register + position bytes */
    int64_t moved_rows;                              /* rows copied by hole-filling compaction so far */
    int64_t attended_keys;                           /* sum over decode steps and units of the live length read */
    int32_t device_status;                           /* most severe device-side error so far (the largest
                                                        corm_status_t code reported), CORM_OK if none. Sticky: once it
                                                        is non-zero, reset the cache (corm_cache_reset) and run the
                                                        prompt pass again before trusting any unit */
    int64_t important_keys;                          /* sum over decode steps and units of the keys judged important
                                                        (Definition 3.1, OR over the group): important_keys /
                                                        attended_keys is the sparsity figure of Section 3.1 */
    int64_t near_threshold;                          /* verdicts (Definition 3.1) whose reduced-precision logit fell
                                                        inside the proven error bound around its threshold and was
                                                        formed again in fp64 before it was decided: only the tiled
                                                        prompt pass places logits in fp32; decode logits are fp64
                                                        throughout and add nothing here */
} corm_stats_t;

/* Bytes of device memory a cache with this configuration needs (host, pure). 0 if the configuration is invalid. */
size_t corm_cache_arena_bytes(const corm_config_t* cfg);

/* Builds the host object over a caller-allocated device arena (256-byte aligned, >= corm_cache_arena_bytes) and
 * zeroes the bookkeeping part of the arena on the legacy default stream, synchronously.
 * Errors: INVALID_ARG (null/invalid fields), UNSUPPORTED (head_dim, group, w > 256), ARENA_TOO_SMALL, CUDA. */
corm_status_t corm_cache_create(const corm_config_t* cfg, void* arena_device, size_t arena_bytes,
                                corm_cache_t** out);

/* Paged variant of the cache (the paper's result is KV memory saved, abstract and Section 5: with one slab of
 * max_tokens rows per unit that saving is only a count; here evicted keys give their memory back). K and V of a
 * layer live in one pool of `pool_pages` pages of 32 keys shared by all units of the layer; a unit holds
 * live / 32 + 1 pages (the last one takes its next append) listed in its page table, claims a page when an append
 * crosses a page boundary and returns pages as its live length shrinks. Registers and positions (8 bytes per key)
 * stay in per-unit arrays of max_tokens entries, and max_tokens still bounds a unit's live length. Every other call
 * works on a paged cache unchanged and gives the same results as on a slab cache; slot order and live lengths are
 * identical too (the page table only changes where a slot's rows are stored).
 *   pool_pages  pages per layer: a multiple of 32, >= batch * n_kv_heads (a unit always owns one page).
 * A pool that runs out: the unit that could not get a page reports CORM_ERR_CAPACITY through the device status at
 * its next decode step and is left untouched from then on, like a unit whose slab is full; a prompt pass whose
 * survivors do not fit reports the same and leaves the unit empty. corm_compress_prompt on a layer returns all of
 * that layer's pages to the pool first.
 * Errors: as corm_cache_create; INVALID_ARG for a bad pool_pages (corm_cache_arena_bytes_paged returns 0). */
size_t corm_cache_arena_bytes_paged(const corm_config_t* cfg, int32_t pool_pages);
corm_status_t corm_cache_create_paged(const corm_config_t* cfg, int32_t pool_pages, void* arena_device,
                                      size_t arena_bytes, corm_cache_t** out);
/* Pages of one layer's pool in use and in total (0 and 0 for a slab cache). Synchronises `stream`. */
corm_status_t corm_cache_pool_usage(corm_cache_t* cache, int32_t layer, int64_t* pages_in_use, int64_t* pages_total,
                                    void* stream);
corm_status_t corm_cache_destroy(corm_cache_t* cache);

/* Empties every unit (asynchronous on `stream`); a prompt pass is needed again before decoding. */
corm_status_t corm_cache_reset(corm_cache_t* cache, void* stream);

/* Prompt-end pass for one layer (the paper covers generation only; this applies Algorithm 1's recording and
 * eviction to the causal attention rows, Eq. 2, of the last min(P, w) prompt queries over the full prompt: the
 * query at position i uses threshold alpha/i, keys newer than a query get a 0 bit as Algorithm 1's zero padding
 * prescribes, and one eviction with t = P follows when w rows exist).
 *   k_prompt, v_prompt  device [batch, n_kv_heads, p_max, head_dim]; rows >= prompt_lens[b] are ignored
 *   q_last              device [batch, n_q_heads, window_w, head_dim]: queries of positions P-w+1..P, oldest
 *                       first; for P < w the first w-P rows are ignored
 *   prompt_lens_host    host [batch], 0 <= P_b <= min(p_max, max_tokens); P_b = 0 leaves the unit empty
 * Survivors are written to the slabs in token order. Produces no attention output. Whatever the layer held
 * before is replaced and its counters (corm_cache_stats) restart. */
corm_status_t corm_compress_prompt(corm_cache_t* cache, int32_t layer, const void* k_prompt, const void* v_prompt,
                                   const void* q_last, const int32_t* prompt_lens_host, int32_t p_max,
                                   void* stream);

/* One decode step of one layer for all sequences (Algorithm 1 around Eq. 1/Eq. 2):
 * appends (k_new, v_new) as token t = tokens_so_far + 1, computes out = softmax(q K^T / sqrt(head_dim)) V over the
 * live keys including the new one, marks each key important iff its probability >= alpha/t for at least one query
 * head of its group, shifts that verdict into the key's register, and, once w verdict rows exist, removes keys
 * whose register is zero and whose position is <= t - r. The output uses the cache before this step's eviction.
 *   q      device [batch, n_q_heads, head_dim]
 *   k_new  device [batch, n_kv_heads, head_dim], v_new likewise
 *   out    device [batch, n_q_heads, head_dim]
 * The call enqueues one or two launches and returns; it sizes them from the longest and the mean live length the
 * kernels last reported, which it reads back asynchronously every 8 steps (batch * n_kv_heads integers). A host that has run 24 steps past a read-back that
 * has not landed waits for it here (the GPU still has those steps queued), so the call can block briefly, and a
 * layer's decode steps cannot be recorded into a CUDA graph.
 * Errors: STATE if the layer has had no corm_compress_prompt since create/reset; INVALID_ARG. */
corm_status_t corm_decode_step(corm_cache_t* cache, int32_t layer, const void* q, const void* k_new,
                               const void* v_new, void* out, void* stream);

/* The same step for n_layers consecutive layers from one host call: layer first_layer + i takes q[i], k_new[i],
 * v_new[i] and writes out[i] (host arrays of device pointers, each as for corm_decode_step). The paper applies the
 * policy "on each head at every layer" (footnote to the Approach paragraph) and the layers of a cache are independent
 * (each has its own token and row counts), so the result is exactly that of n_layers calls of corm_decode_step in
 * layer order on `stream` (outputs within rounding: blocks may be cut differently). It exists because one launch per
 * layer of a single-sequence model is a few microseconds of GPU work behind a chain of launch and memory latencies:
 * when the layers' buffers are contiguous in layer order (q[i + 1] directly behind q[i], likewise k_new, v_new, out),
 * the cache is a slab cache on the bf16 / head_dim-128 kernels, and all the layers are at the same step, ALL layers
 * run as one launch (the layers' units are one array to the kernels); otherwise the per-layer launches are enqueued
 * one after the other. The step's counters are then added to the first layer's (totals in corm_cache_stats are
 * the same). In a model the layers' inputs depend on each other's outputs; use this where they are all known
 * (replay, benchmarking, speculative batches), the per-layer call otherwise.
 * Errors: as corm_decode_step, all arguments and every layer's state checked before anything is enqueued. */
corm_status_t corm_decode_step_layers(corm_cache_t* cache, int32_t first_layer, int32_t n_layers,
                                      const void* const* q, const void* const* k_new, const void* const* v_new,
                                      void* const* out, void* stream);

/* n_steps consecutive decode steps of n_layers consecutive layers from one host call, for callers that hold the
 * inputs of all those steps before the first one runs: scoring a given text (the paper's language-modelling
 * experiments feed known tokens; a layer's queries, keys and values for all positions can be formed before its cache
 * is stepped through them), replay, benchmarking. Buffers are device arrays laid out [n_steps][n_layers] of the
 * per-layer tensors of corm_decode_step:
 *   q, out        [n_steps][n_layers][batch, n_q_heads, head_dim]
 *   k_new, v_new  [n_steps][n_layers][batch, n_kv_heads, head_dim]
 * Every input must be complete in stream order before the call; the result is that of calling corm_decode_step_layers
 * once per step (registers, live lists and positions identical, outputs within rounding).
 * What the call adds: the units of a cache are independent (Algorithm 1 runs "on each head at every layer"), so
 * step s + 1 of a unit needs step s of that unit only. When a step's launch finishes every unit inside the streaming
 * kernel (one query head per KV head; grouped heads inside this call, which take a block per split unless units are
 * few and long; tuning values 2 and 6), the next step's launch is chained to it: its blocks start
 * as soon as a multiprocessor has room and each waits (bounded, like every wait here) for its own unit's previous
 * step instead of the whole previous launch, so consecutive steps fill one another's last waves. Steps that need the
 * verdict launch, and caches with the similarity monitor on, run as with the per-step calls.
 * Errors: as corm_decode_step_layers; n_steps == 0 is a no-op. A failing step leaves the steps before it enqueued. */
corm_status_t corm_decode_steps(corm_cache_t* cache, int32_t first_layer, int32_t n_layers, int32_t n_steps,
                                const void* q, const void* k_new, const void* v_new, void* out, void* stream);

/* corm_decode_steps with HOST buffers of the same layout, asynchronous on `stream`. Pinned, mapped buffers are read
 * and written in place by the kernels (as corm_decode_step_host does); any other host memory goes step by step and
 * layer by layer through the staging buffers. Errors: as corm_decode_steps. */
corm_status_t corm_decode_steps_host(corm_cache_t* cache, int32_t first_layer, int32_t n_layers, int32_t n_steps,
                                     const void* q_host, const void* k_new_host, const void* v_new_host, void* out_host,
                                     void* stream);

/* Same step with HOST buffers, asynchronous on `stream` (out_host is valid once the stream has been synchronised).
 * Pinned buffers the device can address (cudaHostAlloc / cudaHostRegister, 16-byte aligned) are read and written by
 * the kernels directly across the bus, with no copies; any other host memory is copied to staging space inside the
 * arena before the step and out is copied back after it. */
corm_status_t corm_decode_step_host(corm_cache_t* cache, int32_t layer, const void* q_host, const void* k_new_host,
                                    const void* v_new_host, void* out_host, void* stream);

/* corm_decode_step for callers that cannot allocate device memory. (The paper has no counterpart: this is a
 * packaging variant of the same step, not a different method.)
 * Who needs it: code that receives a fixed set of buffers and may not call cudaMalloc or a framework allocator
 * where the step runs, for example a plugin inside a serving runtime whose memory plan was frozen at start-up, or
 * an embedder that gave the cache only room for K, V, registers and positions. corm_decode_step keeps its per-step
 * scratch (this step's logits, the split partial records, the per-unit arrival counters) in the caller's arena;
 * this variant keeps it in a 16 MiB array built into the library, which every GPU that loads the library holds
 * until the process exits. The caller still passes the cache and q / k_new / v_new / out exactly as for
 * corm_decode_step, results are the same, and the two calls may be mixed freely on one cache.
 * It calls no cudaMalloc/cudaFree and no allocating library routine.
 *   Limit: align256(batch*n_q_heads*max_tokens*8) + align256(batch*n_kv_heads*ceil(live_bound/256)*group*
 *   (16 + 4*head_dim)) + align256(batch*n_kv_heads*4) bytes must fit in 16 MiB (live_bound = the longest prompt so
 *   far + decode steps so far + 1, capped at max_tokens); otherwise CORM_ERR_CAPACITY is returned, a message
 *   naming both sizes goes to stderr and nothing is enqueued.
 *   First call on a device: looks up the array's device address (once per device, that device made current for
 *   the lookup). Make this first call outside any stream capture.
 *   Sharing: all caches and all calls on a device use the same array. It keeps the previous call's contents; the
 *   arrival counters are cleared on `stream` at the start of every call, everything else is rewritten before it
 *   is read. Two calls of this function that overlap on the GPU (different streams, no ordering) race on the
 *   array and give wrong results: keep them stream-ordered.
 * Errors otherwise as corm_decode_step. */
corm_status_t corm_decode_step_static(corm_cache_t* cache, int32_t layer, const void* q, const void* k_new,
                                      const void* v_new, void* out, void* stream);

/* Totals over all units ("compression rate" of Section 5). Synchronises `stream`. */
corm_status_t corm_cache_stats(corm_cache_t* cache, corm_stats_t* out_host, void* stream);

/* Live length of every unit of one layer: live_host [batch, n_kv_heads]. Synchronises `stream`. */
corm_status_t corm_cache_live_lens(corm_cache_t* cache, int32_t layer, int32_t* live_host, void* stream);

/* Test / checkpoint hooks. Host buffers hold max_tokens entries; entries come in SLOT order (see above).
 * k_host, v_host: [max_tokens, head_dim] in kv_dtype; word_host, pos_host: [max_tokens]; scalars by pointer.
 * n_tokens / n_obs are per (layer, sequence): tokens seen and verdict rows recorded (<= w). Synchronise `stream`. */
corm_status_t corm_cache_export_state(corm_cache_t* cache, int32_t layer, int32_t seq, int32_t kv_head,
                                      void* k_host, void* v_host, uint32_t* word_host, int32_t* pos_host,
                                      int32_t* live_len, int32_t* n_tokens, int32_t* n_obs, void* stream);
corm_status_t corm_cache_import_state(corm_cache_t* cache, int32_t layer, int32_t seq, int32_t kv_head,
                                      const void* k_host, const void* v_host, const uint32_t* word_host,
                                      const int32_t* pos_host, int32_t live_len, int32_t n_tokens, int32_t n_obs,
                                      void* stream);

/* Tuning knobs (performance only; live lists and registers do not depend on them, outputs only within rounding):
 * keys per split of the block-per-split decode kernel (multiple of 32, 0 = automatic) and which kernels may be used:
 * allow_fast_path 0 = the generic kernels only; 1 = automatic (default): for bf16 / head_dim 128, one query head per
 * KV head takes the block-per-split kernel, which finishes a unit of several splits inside the decode launch when the
 * launch has many units and by a second, verdict launch when it has few, and grouped heads take the balanced
 * kernel (every block an equal share of the step's keys) followed by the verdict launch; 2 / 3 = the block-per-split
 * kernel with the first / the second way always; 4 / 5 = the balanced kernel for every group size it covers,
 * finishing inside its own launch / with the verdict launch; 6 = the balanced kernel's streaming loop with a block per
 * split, each unit finished by its last-arriving split (what automatic picks for grouped heads inside
 * corm_decode_steps unless units are few and long, because such launches can be chained). Errors: INVALID_ARG. */
corm_status_t corm_cache_set_tuning(corm_cache_t* cache, int32_t split_len, int32_t allow_fast_path);

/* Opt-in monitor of the method's premise (Sections 3.2-3.3: the current query resembles recent ones, which is what
 * lets recent verdicts stand in for future ones, and which the paper reports failing for some models): while
 * enabled, every decode step also forms Eq. 3's cosine similarity between each query head's query and that head's
 * query of the previous decode step of the same layer (one small extra launch per step; the first step after a
 * prompt pass or after enabling has no partner; zero vectors are skipped). corm_cache_similarity returns the sum
 * and the number of pairs since create/reset over all layers and synchronises `stream`. Off by default. */
corm_status_t corm_cache_set_similarity_monitor(corm_cache_t* cache, int32_t enabled);
corm_status_t corm_cache_similarity(corm_cache_t* cache, double* sum_host, int64_t* count_host, void* stream);

/* The tiled prompt pass (bf16, head_dim 128) places each logit of its second launch on one side of its exact
 * threshold with an fp32 dot product wherever a proven bound on the fp32 accumulation error allows, and forms the
 * logit again in fp64 where it does not, so results never depend on this. `scale` >= 1 multiplies the bound
 * (default 1): larger values send more logits through the exact path, which is how the tests exercise it.
 * Errors: INVALID_ARG. */
corm_status_t corm_cache_set_bound_scale(corm_cache_t* cache, double scale);

/* Number of kernels this library has launched on behalf of `cache` since create. */
int64_t corm_cache_kernel_launches(const corm_cache_t* cache);

/* How many of them were chained to the previous step's launch (corm_decode_steps). */
int64_t corm_cache_chained_launches(const corm_cache_t* cache);

const char* corm_status_string(corm_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* CORM_H_ */
