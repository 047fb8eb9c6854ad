/*
 * qevict.h -- C ABI of the B200 decode hot path of a three-tier, window-granular KV cache.
 *
 * What the library computes (paper sections in brackets):
 *   - per (sequence, layer) the historical KV cache is cut into windows of W tokens; every window is
 *     Full (stored in the execution datatype), Quantized (stored as low-bit codes, still attended
 *     to) or Evicted (gone for good)                         [Methodology: Preliminaries, Recoverable
 *                                                             Cache Hierarchy]
 *   - a decode step is softmax attention of one query per head over the accessible tokens only,
 *     grouped-query heads sharing a KV head                  [Preliminaries, attention equation]
 *   - each step adds to every window the attention probability mass its tokens received, summed
 *     over the query heads (the cumulative window score)      [Eq. 1]
 *   - a routing event ranks the candidate windows by score and keeps the best K_f Full, the next
 *     K_q Quantized and deletes the rest; a window is quantized only on its first demotion, a
 *     promotion rebuilds it from its codes, a later demotion reuses the codes  [Dynamic Routing and
 *                                                             Recovery; Migration-Stable
 *                                                             Quantization; Algorithm 1]
 *   - K_f and K_q follow from a byte budget                   [tier-capacity equation; memory
 *                                                             accounting appendix]
 *
 * Conventions
 *   - Every pointer argument says "device" or "host".  Device pointers must be valid on the device
 *     named in the configuration, 16-byte aligned and contiguous; the caller owns them, the library
 *     neither frees nor keeps them after the enqueued work has run.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls only
 *     enqueue work unless the comment says "synchronises".
 *   - A "unit" is one (layer, sequence) pair; unit = layer * batch + sequence.  `layer == -1` means
 *     every layer in one launch; tensors then carry a leading [n_layers] dimension.
 *   - Errors are returned as qevict_status; a call refused for its arguments or its place in the call order
 *     enqueues nothing.  If a CUDA launch fails after an earlier kernel of the same call has been enqueued,
 *     the cache is marked broken and every later compute call on it returns QEVICT_ERR_BAD_STATE.  Kernels
 *     never trap: device-side checks record a code that qevict_get_stats reports as
 *     QEVICT_ERR_DEVICE_CHECK.
 *   - Every call makes the cache's device current while it runs and puts the caller's current device back
 *     before it returns.
 *   - Process-wide state is limited to three things, none of which a caller can observe through results:
 *     the text qevict_last_error(NULL) returns (per thread: the last failure of qevict_create or
 *     qevict_workspace_bytes, which have no handle to keep it in); the per-device record of the
 *     shared-memory limits already granted to the kernels (only ever raised); and the built-in scratch
 *     array of qevict_decode_attn_noalloc with its per-device address.  One handle must not be used from
 *     two threads at once; different handles may be.
 *   - There is no CPU fallback: without a CUDA device every compute call returns QEVICT_ERR_CUDA.
 */
#ifndef QEVICT_H_
#define QEVICT_H_

#include <stdint.h>

#if defined(__GNUC__)
#define QEVICT_API __attribute__((visibility("default")))
#else
#define QEVICT_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct qevict_ctx* qevict_handle;

typedef enum {
  QEVICT_OK = 0,
  QEVICT_ERR_INVALID_ARG = 1,  /* null pointer, out-of-range value, inconsistent configuration */
  QEVICT_ERR_BAD_STATE = 2,    /* call order: decode before prefill, prefill twice, rebalance overdue */
  QEVICT_ERR_NO_MEMORY = 3,    /* caller's device buffer too small, or host allocation failed */
  QEVICT_ERR_UNSUPPORTED = 4,  /* a shape the kernels are not built for */
  QEVICT_ERR_CUDA = 5,         /* a CUDA runtime call failed (qevict_last_error has the text) */
  QEVICT_ERR_DEVICE_CHECK = 6  /* a kernel recorded an internal check failure */
} qevict_status;

enum { QEVICT_DTYPE_FP16 = 0, QEVICT_DTYPE_BF16 = 1 };

/* window states, as exported by qevict_export_tables */
enum {
  QEVICT_TIER_NONE = 0,    /* window index not created yet */
  QEVICT_TIER_OPEN = 1,    /* recent region: the window being filled by appended tokens */
  QEVICT_TIER_AGED = 2,    /* filled: inside the protected recent region, or out of it and waiting for the
                              next routing event */
  QEVICT_TIER_FULL = 3,
  QEVICT_TIER_QUANT = 4,
  QEVICT_TIER_EVICTED = 5,
  QEVICT_TIER_SINK = 6     /* protected sink prefix: full precision, never a candidate */
};
/* ranking functions.  CUMULATIVE is Eq. 1 (mass added to the score at every step).  With the other two
 * the mass is collected in an event accumulator u and folded into the score by every routing event after
 * prefill, for every stored window, in float32 with each operation rounded on its own:
 *   DECAYED  S <- lambda * S + u;   PNORM  P <- P + u^p (p - 1 multiplications); windows are ranked by
 *   P, which orders them as S_p = P^(1/p) does.  The prefill scores initialise S (or P) directly.
 * KEYNORM is attention-free: the score of a window is minus the mean L2 norm of its keys (per KV head, averaged
 * over heads and tokens), fixed when the window is complete; window_scores of qevict_prefill_assign is
 * ignored and may be NULL; the attention mass is still collected in u but never enters the score. */
enum { QEVICT_RANK_CUMULATIVE = 0, QEVICT_RANK_DECAYED = 1, QEVICT_RANK_PNORM = 2, QEVICT_RANK_KEYNORM = 3 };
/* ledger states */
enum { QEVICT_LEDGER_NONE = 0, QEVICT_LEDGER_ACTIVE = 1, QEVICT_LEDGER_DORMANT = 2 };

typedef struct {
  uint32_t struct_size;      /* sizeof(qevict_config) of the caller, for ABI growth */
  int32_t batch;             /* sequences per layer */
  int32_t n_layers;
  int32_t n_q_heads;         /* H_q */
  int32_t n_kv_heads;        /* H_kv; H_q % H_kv == 0 and H_q / H_kv <= 8 */
  int32_t head_dim;          /* d: 64 or 128 */
  int32_t dtype;             /* QEVICT_DTYPE_* : execution datatype of q, k, v, out */
  int32_t window;            /* W tokens: 32 or 64 */
  int32_t quant_bits;        /* b: 2 or 4 */
  int32_t group_size;        /* g: 32 or 64; W % g == 0 and d % g == 0 */
  int32_t fp_budget_windows; /* K_f per unit */
  int32_t q_budget_windows;  /* K_q per unit */
  int32_t max_context;       /* upper bound on prompt + generated tokens; multiple of W */
  int32_t rebalance_interval_hint; /* decode steps the caller lets pass between routing events; sizes
                                      the full-precision pages that hold aged windows; 0 => W */
  float softmax_scale;       /* 0 => 1/sqrt(d) */
  int32_t device;            /* CUDA device ordinal */
  int32_t sink_windows;      /* protected sink prefix: the first windows of the prompt stay in full precision,
                                are never candidates and do not count against K_f [cache partition] */
  int32_t recent_windows;    /* protected recent region: besides the window being filled, this many of the
                                most recently filled windows stay in full precision and are not candidates
                                until newer windows push them out [candidate pool: windows that have exited
                                the recent region] */
  int32_t rank_mode;         /* QEVICT_RANK_*: which score orders the candidates [ranking-function appendix] */
  float rank_param;          /* lambda of the decayed score (0 < lambda <= 1); p of the p-norm (integer 2..8) */
  int32_t one_way;           /* 1: no promotion [promotion ablation: Full -> Quantized -> Evicted].  The paper gives
                                only the transition diagram; reading: the Full tier is the best K_f candidates that
                                are not Quantized, the Quantized tier the best K_q of all the others.  0: Algorithm 1 */
  float rope_base;           /* > 0: the keys handed to the cache (prompt and k_new) are pre-RoPE and stay so in every
                                tier; the attention kernel rotates each key for its absolute position (slot j of
                                window w is position w * W + j) when it reads it, after dequantization for the
                                low-bit tier [Migration-Stable Quantization: keys in the pre-RoPE domain with their
                                absolute positions, RoPE reapplied after dequantization].  theta_i = rope_base^(-2i/d),
                                pairs (i, i + d/2); cos, sin and every product and sum rounded to the execution
                                datatype, as the models' own implementation does.  q arrives rotated.  0: keys are
                                used as given. */
} qevict_config;

typedef struct {
  uint64_t promotions;     /* Quantized -> Full (dequantize into a full-precision page) */
  uint64_t quantizations;  /* first demotions: the only time a window's codes are produced */
  uint64_t reactivations;  /* Full -> Quantized with a dormant ledger entry: no data moved */
  uint64_t deletions;      /* windows evicted */
  uint64_t n_full, n_quant, n_aged, n_open, n_evicted; /* current window counts */
  uint64_t decode_steps;
  uint64_t n_sink;         /* protected sink windows */
} qevict_stats;

/* Bytes of one Full window and one Quantized window (all KV heads, keys and values), and the tier
 * capacities K_f = floor((1-q_frac) * hist_bytes / M_f), K_q = floor(q_frac * hist_bytes / M_q)
 * [tier-capacity equation].  M_q counts packed codes plus one (scale, zero) pair of the execution
 * datatype per group [memory accounting appendix].  hist_bytes is the historical budget: what is left of the
 * total after the protected regions, (sink_windows + recent_windows + 1) * M_f, have been set aside [budget
 * constraint: B_sink + B_local + the tiers <= B_total].  Host arithmetic only; any output pointer may be
 * NULL.  Only the shape fields of `cfg` are read. */
QEVICT_API qevict_status qevict_budget_from_bytes(const qevict_config* cfg, uint64_t hist_bytes, double q_frac,
                                       int32_t* k_f, int32_t* k_q, uint64_t* m_f, uint64_t* m_q);

/* Size of the device buffer qevict_create needs for this configuration (pools, tables, scratch).
 * QEVICT_ERR_UNSUPPORTED for shapes the kernels are not built for: head_dim other than 64 / 128, window other
 * than 32 / 64, more than 8 query heads per KV head, more than 8192 windows per sequence, budgets whose decode
 * work list (K_f + K_q + protected windows + waiting windows + 1) exceeds 8192 entries, routing tables that do
 * not fit the shared memory of an SM; qevict_last_error(NULL) says which. */
QEVICT_API qevict_status qevict_workspace_bytes(const qevict_config* cfg, uint64_t* bytes);

/* Build a cache inside `device_mem` (device pointer, 256-byte aligned, `bytes` long, owned by the
 * caller and kept alive until qevict_destroy).  Clears the tables; synchronises the device once.
 * The memory is fixed from here on: the pools hold K_f + aged + 1 full-precision pages and
 * K_q + K_f quantized pages per unit (the extra K_f keep the codes of promoted windows). */
QEVICT_API qevict_status qevict_create(const qevict_config* cfg, void* device_mem, uint64_t bytes, qevict_handle* out);
QEVICT_API qevict_status qevict_destroy(qevict_handle h);

/* Prefill initialisation [Methodology: prompt attention initialises the window scores and the first
 * tier assignment].  For every sequence of `layer`: the prompt is cut into ctx_tokens / W windows,
 * window w starts with score window_scores[seq][w], one routing event runs, Full windows are copied
 * and Quantized windows are quantized straight from the prompt, the rest is never stored.
 *   k, v          device, [batch][H_kv][ctx_tokens][d] in the execution datatype ([n_layers][...] first
 *                 when layer == -1)
 *   window_scores device, float32 [batch][ctx_tokens / W]: raw attention mass summed over heads
 *   ctx_tokens    multiple of W, at most max_context
 * Once per layer. */
QEVICT_API qevict_status qevict_prefill_assign(qevict_handle h, int32_t layer, const void* k, const void* v,
                                    int32_t ctx_tokens, const float* window_scores, void* stream);

/* Prefill window scores computed on the GPU [Methodology: prompt attention initialises the window scores;
 * Eq. 1's form].  For every sequence of one layer, n_obs observation queries per query head -- queries that
 * stand after the prompt, e.g. its last n_obs positions' queries -- attend over the whole prompt in full
 * precision, and
 *     window_scores[seq][w] = sum over observation queries and query heads of the softmax mass of window w
 * (raw sum, the input qevict_prefill_assign expects).  Which queries observe is the caller's choice: the paper
 * does not fix it.
 *   k             device, [batch][H_kv][ctx_tokens][d] in the execution datatype (one layer)
 *   q_obs         device, [batch][n_obs][H_q][d], n_obs in 1..64
 *   window_scores device, float32 [batch][ctx_tokens / W] (output)
 *   scratch       device, at least qevict_prefill_score_scratch_bytes(...) bytes, 16-byte aligned; contents
 *                 are overwritten
 * With rope_base > 0 the keys are pre-RoPE like everything the cache is given: the scores are taken over a copy
 * rotated for positions 0 .. ctx_tokens - 1, kept in the scratch buffer (which is that much larger).
 * Deterministic (fixed summation order). */
QEVICT_API qevict_status qevict_prefill_score_scratch_bytes(qevict_handle h, int32_t n_obs, int32_t ctx_tokens,
                                                            uint64_t* bytes);
QEVICT_API qevict_status qevict_prefill_score(qevict_handle h, const void* k, const void* q_obs, int32_t n_obs,
                                              int32_t ctx_tokens, float* window_scores, void* scratch,
                                              uint64_t scratch_bytes, void* stream);

/* One decode step [attention equation; Eq. 1].  If k_new != NULL the new token's key and value
 * first enter the recent region (the open window); then every query head attends over all accessible
 * tokens (open, aged, Full and Quantized windows, the latter dequantized in registers) and each
 * window's score grows by the probability mass it received, summed over the query heads.
 *   q            device, [batch][H_q][d]
 *   k_new, v_new device, [batch][H_kv][d], or both NULL (fixed context)
 *   out          device, [batch][H_q][d]
 * Returns QEVICT_ERR_BAD_STATE if more filled windows are waiting than the pages sized by
 * rebalance_interval_hint can hold (call qevict_rebalance first). */
QEVICT_API qevict_status qevict_decode_attn(qevict_handle h, int32_t layer, const void* q, const void* k_new,
                                 const void* v_new, void* out, void* stream);

/* The same step with HOST buffers (pageable or page-locked): brings q, k_new, v_new to the device, runs the
 * step, returns `out` to the host and synchronises the stream.  q always ends up in device memory before the
 * attention kernel runs (every CTA of that kernel reads it).  Page-locked buffers the device can address (any
 * cudaHostAlloc / cudaHostRegister memory under unified addressing) need no copy operation at all: the append
 * kernel reads k_new and v_new from them in place and, in the same launch, brings q into the cache's staging
 * buffer; the merge kernel writes `out` into the host buffer over the bus.  Pageable buffers, and q when there
 * is no new token, take staged copies.  The bytes that cross the bus are the same either way. */
QEVICT_API qevict_status qevict_decode_attn_host(qevict_handle h, int32_t layer, const void* q_host,
                                      const void* k_new_host, const void* v_new_host, void* out_host,
                                      void* stream);

/* The same without the final synchronisation: the copies and the step are only enqueued.  `out_host` holds
 * the result once the caller has synchronised `stream`; the host buffers must stay valid and unchanged until
 * then (pinned memory, or the copies are not asynchronous).  Lets the caller enqueue more work -- the
 * step's routing event, for one -- before it waits for the result. */
QEVICT_API qevict_status qevict_decode_attn_host_async(qevict_handle h, int32_t layer, const void* q_host,
                                                       const void* k_new_host, const void* v_new_host,
                                                       void* out_host, void* stream);

/* Blocks the calling thread until the `out_host` of this cache's most recent qevict_decode_attn_host_async call is
 * complete in host memory -- and no longer: work enqueued behind that call (the step's routing event, say) keeps
 * running.  The call records an event behind the last operation that writes `out_host`; this waits for it.
 * QEVICT_ERR_BAD_STATE if no such call has been made. */
QEVICT_API qevict_status qevict_wait_result(qevict_handle h);

/* The same decode step for callers that must not allocate device memory (the paper has no counterpart:
 * this is a deployment variant of qevict_decode_attn, not a step of the method).
 *
 * Who needs it: code that runs under a fixed device-memory plan.  A serving process that hands all of
 * HBM to its own pool at start-up has nothing left for a library to allocate from; a latency-critical
 * thread must not enter the CUDA allocator, which can block behind other work on the device.  Such a
 * caller can still build a cache inside memory it already owns (qevict_create takes the buffer), but the
 * attention kernel also wants scratch for its per-split partial results.  This entry point keeps that
 * scratch in a fixed array of QEVICT_NOALLOC_SCRATCH_BYTES that is part of the library's device image:
 * every GPU that loads the library holds those bytes until the process exits, and nothing is allocated
 * or freed by the call (no cudaMalloc / cudaFree, no allocating library routine).
 *
 * Arguments, results and state changes are those of qevict_decode_attn.  Differences:
 *   - A call whose scratch (the partials of the units of THIS call: one layer's sequences, or all of them
 *     with layer == -1) does not fit the array returns QEVICT_ERR_NO_MEMORY and enqueues nothing;
 *     qevict_last_error states the size needed.
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress) before it
 *     launches anything.  Where the CUDA runtime loads modules lazily, that look-up is also the moment the
 *     runtime places the library's device image -- the array included -- in device memory, so the first
 *     call can fail with an out-of-memory error on a device whose memory has already been handed out in
 *     full: make it once at start-up, before the memory plan is committed and before any stream capture
 *     begins.  Later calls allocate nothing.
 *   - qevict_set_kernel_timing does not cover this entry point (its launches are not bracketed by events).
 *   - All calls, on all handles and streams of a device, share the one array, which keeps the last
 *     call's contents.  Nothing in it has to start at zero -- every slot a call reads it has written
 *     first -- but two calls that overlap on the GPU race on it: keep them in one stream, or order them
 *     with events. */
#define QEVICT_NOALLOC_SCRATCH_BYTES (8u << 20)
QEVICT_API qevict_status qevict_decode_attn_noalloc(qevict_handle h, int32_t layer, const void* q, const void* k_new,
                                                    const void* v_new, void* out, void* stream);

/* One routing event [Algorithm 1].  Candidates = Full, Quantized and aged windows, ranked by score
 * (float32, higher first, lower window index first among equals); the first K_f become Full, the next
 * K_q Quantized, the rest Evicted.  Pages are released, then handed out in ascending page id to the
 * windows that need one in ascending window index; first demotions are quantized, promotions are
 * dequantized (after the quantizations, because a promotion may receive a page a demotion released);
 * a demotion with a dormant ledger entry only flips its flag. */
QEVICT_API qevict_status qevict_rebalance(qevict_handle h, int32_t layer, void* stream);

/* Counters of one layer (layer == -1: all layers), summed over its sequences.  Synchronises. */
QEVICT_API qevict_status qevict_get_stats(qevict_handle h, int32_t layer, qevict_stats* out);

/* Synchronises the device and reports the device status word: QEVICT_OK, or QEVICT_ERR_DEVICE_CHECK if a kernel
 * of this cache has recorded a failed internal check since creation (pool exhausted, work list longer than the
 * host's bound, a page copy that did not arrive in time; in the checking build also an index out of range).
 * *code (may be NULL) receives the recorded code, 0 if none; the first failure is the one kept.  The same report
 * comes with qevict_get_stats. */
QEVICT_API qevict_status qevict_check_device(qevict_handle h, int32_t* code);

/* Tables of one unit, written to DEVICE buffers sized for max_context / W windows (any may be NULL):
 * n_windows int32[1], tier uint8[], ledger uint8[], fp_page int32[], q_page int32[] (-1 = none),
 * importance float32[].  Enqueues only. */
QEVICT_API qevict_status qevict_export_tables(qevict_handle h, int32_t layer, int32_t seq, int32_t* n_windows,
                                   uint8_t* tier, uint8_t* ledger, int32_t* fp_page, int32_t* q_page,
                                   float* importance, void* stream);

/* Attention mass of the last decode step per window, DEVICE float32[max_context / W] (0 where the
 * window was not attended). */
QEVICT_API qevict_status qevict_export_last_mass(qevict_handle h, int32_t layer, int32_t seq, float* mass, void* stream);

/* Contents of the full-precision page `fp_page` of a unit in plain layout: DEVICE k_out, v_out
 * [H_kv][W][d] in the execution datatype. */
QEVICT_API qevict_status qevict_export_fp_page(qevict_handle h, int32_t layer, int32_t seq, int32_t fp_page,
                                    void* k_out, void* v_out, void* stream);

/* Contents of the quantized page `q_page` of a unit in plain layout, DEVICE buffers:
 * k_codes, v_codes uint8 [H_kv][W][d] (one code per byte);
 * k_params [H_kv][W/g][d][2], v_params [H_kv][W][d/g][2] in the execution datatype, (scale, zero). */
QEVICT_API qevict_status qevict_export_q_page(qevict_handle h, int32_t layer, int32_t seq, int32_t q_page,
                                   uint8_t* k_codes, void* k_params, uint8_t* v_codes, void* v_params,
                                   void* stream);

/* The event accumulator u of a unit (rank_mode DECAYED or PNORM): float32 [max_context / W], DEVICE
 * buffer; all zeros right after a routing event. */
QEVICT_API qevict_status qevict_export_event_mass(qevict_handle h, int32_t layer, int32_t seq, float* event_mass,
                                                  void* stream);

/* Snapshot and restore of one unit [Migration-Stable Quantization: the ledger is a persistent low-bit store;
 * codes written at a window's first demotion stay valid for the window's whole life, so a cache can be put
 * away and brought back without requantizing anything].  A snapshot holds what the kernels read for one
 * (layer, sequence) pair -- window tables, page-owner tables, decode work list, the unit's pages of both pools
 * and the host's bookkeeping for the layer -- and restores into any cache created with the same
 * configuration, after which decode steps and routing events continue bit for bit as they would have.
 *
 * All arrays are HOST memory owned by the caller, sized by qevict_state_layout_of:
 *   tier, ledger uint8 [n_window_slots]; fp_page, q_page int32 [n_window_slots] (-1 = none); importance,
 *   event_mass float32 [n_window_slots]; fp_owner int32 [n_fp_pages], q_owner int32 [n_q_pages] (window that
 *   holds the page, -1 = free); entries uint32 [n_entries][2] ({window | kind << 28, page}; kind 0 full
 *   precision, 1 quantized, 2 open window); last_mass float32 [n_entries] (mass of the last decode step per
 *   work-list entry); fp_pool [fp_pool_bytes], q_pool [q_pool_bytes]: the unit's pages in the library's own
 *   page layout (opaque; use qevict_export_fp_page / qevict_export_q_page for plain layouts).
 * qevict_export_state synchronises the device, fills the scalars and the arrays.  qevict_import_state checks
 * every index in the snapshot against the configuration (a snapshot that fails a check changes nothing),
 * synchronises the device and overwrites the unit.  The sequences of a layer step together, so the layer's
 * bookkeeping (windows, fill of the open window, filled windows waiting for a routing event) is taken from the
 * first snapshot imported into a layer that has not been prefilled, and every later import into that layer
 * must agree with it (QEVICT_ERR_BAD_STATE otherwise); import every sequence of a layer before using it. */
typedef struct {
  int32_t n_window_slots;  /* max_context / W */
  int32_t n_fp_pages;      /* full-precision pages per unit */
  int32_t n_q_pages;       /* quantized pages per unit */
  int32_t n_entries;       /* capacity of the decode work list */
  uint64_t fp_pool_bytes;  /* n_fp_pages * bytes of a full-precision page */
  uint64_t q_pool_bytes;   /* n_q_pages * bytes of a quantized page */
} qevict_state_layout;

typedef struct {
  uint32_t struct_size;    /* sizeof(qevict_state_view) of the caller */
  int32_t n_windows;       /* windows created so far */
  int32_t open_window;     /* index of the window being filled, -1 if none */
  int32_t open_fill;       /* tokens in it */
  int32_t n_live;          /* entries of the decode work list */
  int32_t layer_prefilled, layer_has_open, layer_open_fill, layer_n_windows, layer_aged; /* host bookkeeping of the layer */
  float knorm_acc;         /* key-norm ranking: running sum of the open window */
  uint64_t counters[4];    /* promotions, quantizations, reactivations, deletions of the unit */
  uint64_t decode_steps;   /* of the handle */
  uint8_t* tier;
  uint8_t* ledger;
  int32_t* fp_page;
  int32_t* q_page;
  float* importance;
  float* event_mass;
  int32_t* fp_owner;
  int32_t* q_owner;
  uint32_t* entries;
  float* last_mass;
  void* fp_pool;
  void* q_pool;
} qevict_state_view;

QEVICT_API qevict_status qevict_state_layout_of(qevict_handle h, qevict_state_layout* out);
QEVICT_API qevict_status qevict_export_state(qevict_handle h, int32_t layer, int32_t seq, qevict_state_view* view);
QEVICT_API qevict_status qevict_import_state(qevict_handle h, int32_t layer, int32_t seq, const qevict_state_view* view);

/* Tuning: force the number of KV splits per (unit, KV head) of the decode kernel (1..64); 0 restores
 * the built-in choice, which fills the GPU in whole waves.  Results do not depend on it beyond
 * floating-point summation order. */
QEVICT_API qevict_status qevict_set_splits(qevict_handle h, int32_t splits);

/* Instrumentation: while enabled, every kernel of the decode and rebalance calls is bracketed with CUDA
 * events on the call's stream.  qevict_kernel_time synchronises on the recorded events, returns the
 * summed duration in milliseconds and the launch count of the attention kernel (the dominant kernel of
 * the path), and forgets all recorded events; qevict_kernel_times does the same for every kernel:
 * index 0 append, 1 attention, 2 combine, 3 route, 4 migrate (arrays of QEVICT_N_KERNELS). */
enum { QEVICT_N_KERNELS = 5 };
QEVICT_API qevict_status qevict_set_kernel_timing(qevict_handle h, int32_t enable);
QEVICT_API qevict_status qevict_kernel_time(qevict_handle h, double* total_ms, uint64_t* n_launches);
QEVICT_API qevict_status qevict_kernel_times(qevict_handle h, double* total_ms, uint64_t* n_launches);

/* Kernel timeline (tracing build of the library only: the same sources compiled with -DQEVICT_TRACE, in which
 * every warp of the five step kernels stamps the GPU's nanosecond timer when it starts and when it ends).
 * Synchronises the device and returns the launches made since the previous call of this function (those of the
 * first 512 API calls; later ones are not recorded), oldest first, the most recent max_records of them:
 * kernel[i] (0 append, 1 attention, 2 combine, 3 route, 4 migrate), start_us[i] = earliest warp start and
 * end_us[i] = latest warp end, in microseconds from the first returned start (host arrays of max_records);
 * *n_records = how many were written.  Then clears the record.  Unlike CUDA events around a launch, this sees
 * the kernels inside the running pipeline, where the next kernel's launch overlaps the current one.
 * QEVICT_ERR_UNSUPPORTED (and *n_records = 0) in the normal build. */
QEVICT_API qevict_status qevict_kernel_timeline(qevict_handle h, int32_t max_records, int32_t* kernel, double* start_us,
                                                double* end_us, int32_t* n_records);

/* Number of kernels this handle has launched since creation (host counter). */
QEVICT_API uint64_t qevict_launch_count(qevict_handle h);

/* Text of the last error on this handle (never NULL).  With h == NULL: the calling thread's last failure of
 * qevict_create or qevict_workspace_bytes. */
QEVICT_API const char* qevict_last_error(qevict_handle h);
QEVICT_API const char* qevict_status_string(qevict_status s);
/* Library version, "major.minor". */
QEVICT_API const char* qevict_version(void);
/* Which build of the sources this library is: 0 the normal one; 1 the tracing build (-DQEVICT_TRACE: kernel
 * timeline); 2 the checking build (-DQEVICT_DEBUG_BOUNDS: every page id, window index, work-list entry and
 * migration record a kernel reads from a table is range-checked before use -- a value out of range is recorded
 * (qevict_get_stats then returns QEVICT_ERR_DEVICE_CHECK with the code in qevict_last_error) and the access is
 * skipped, nothing traps -- and both pools start filled with a NaN pattern so that a read of a page nobody wrote
 * shows in the results).  The checking build stands in for a memory checker; it computes the same results. */
QEVICT_API int32_t qevict_build_flavour(void);

#ifdef __cplusplus
}
#endif
#endif /* QEVICT_H_ */
