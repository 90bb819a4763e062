/*
 * crystalkv.h — C ABI of the Crystal-KV decode hot path for NVIDIA B200 (sm_100a).
 *
 * One handle owns, on one GPU, the compressed KV cache of `batch` independent
 * sequences of a GQA transformer: a pool of K/V pages (16 entries each) per sequence,
 * per (sequence, layer, kv head) a page table and the entries' CRF / last-hit-time
 * metadata, and the per-head budgets.  Notation follows the paper: B budget, p top-p threshold, lambda
 * CRF decay, t time step, tau last hit time, CRF the combined recency-frequency score.
 *
 * Conventions
 *   - Tensors are dense, row-major, bf16 (2 bytes per element), head_dim = 128.
 *   - "dev" pointers are device memory on the handle's GPU, "host" pointers are host
 *     memory.  The caller owns every pointer it passes; the library owns the pool,
 *     the lists and the metadata and frees them in crystalkv_destroy.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Work is enqueued on it; hot-path calls neither synchronise the host nor allocate.
 *     The Algorithm 1 part of a decode step runs on a stream the handle owns, ordered
 *     behind the step's attention by an event; later calls order themselves behind it.
 *   - Every call returns 0 on success or a negative CRYSTALKV_E* code; nothing throws
 *     or aborts across this boundary.  crystalkv_strerror() gives the text of a code,
 *     crystalkv_last_error() the detail of the handle's most recent failure.
 *   - A handle is not thread-safe and is used with one stream at a time.
 */
#ifndef CRYSTALKV_H
#define CRYSTALKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CRYSTALKV_OK 0
#define CRYSTALKV_EINVAL (-1)   /* null pointer, value out of range, unsupported dtype / head_dim */
#define CRYSTALKV_ESTATE (-2)   /* call out of order, capacity or context exhausted */
#define CRYSTALKV_ENOMEM (-3)   /* device allocation failed */
#define CRYSTALKV_ECUDA (-4)    /* CUDA runtime error (sticky for the handle) */
#define CRYSTALKV_ECHECK (-5)   /* a device-side consistency check raised the handle's error word */

#define CRYSTALKV_BF16 1

#define CRYSTALKV_MODE_EVICT 0   /* Algorithm 1 runs every think step */
#define CRYSTALKV_MODE_FULLKV 1  /* FullKV baseline of Section 6.1: nothing tracked, nothing evicted */

#define CRYSTALKV_STAGE_THINK 0
#define CRYSTALKV_STAGE_ANSWER 1

typedef struct crystalkv crystalkv_t;

typedef struct {
  int32_t n_layers;        /* L */
  int32_t n_q_heads;       /* multiple of n_kv_heads; group size G = n_q_heads / n_kv_heads <= 8 */
  int32_t n_kv_heads;      /* H */
  int32_t head_dim;        /* 128 */
  int32_t batch;           /* independent sequences, each with its own budgets (Algorithm 2 is per inference) */
  int32_t dtype;           /* CRYSTALKV_BF16 */
  int32_t budget_per_head; /* B_total per sequence = budget_per_head * L * H (Algorithm 2 input) */
  int32_t min_budget;      /* floor of a head's budget under reallocation; 0 = max(16, budget_per_head / 8) */
  int32_t max_budget;      /* cap of a head's budget; 0 = 4 * budget_per_head; >= budget_per_head */
  int32_t max_answer_tokens; /* entries a head may append beyond its budget in the answer stage */
  int32_t max_context;     /* largest token position + 1; sizes the lambda^D table and FullKV capacity */
  float top_p;             /* hit threshold p in (0, 1]; 0 = 0.9 (Section 6.4) */
  float lambda;            /* CRF decay in [0, 1]; negative = 0.6 (Section 6.4) */
  float sm_scale;          /* logit scale; 0 = 1/sqrt(head_dim) */
  int32_t mode;            /* CRYSTALKV_MODE_* */
  int32_t device;          /* CUDA device ordinal */
  int32_t evict_every;     /* m: Algorithm 1 step 4 waits until a head is m entries over its budget and then
                              removes all of them in one call (k = m); 0 or 1 = every step.  At most 4096. */
  int32_t literal_return;  /* 1: Algorithm 1's first line as printed: while Len(K) < B of a head nothing
                              of the algorithm runs for it (no hit mask, no CRF update); 0 = track always */
  float budget_ratio;      /* r > 0: ratio budgets (Section 6.1, Table 1's "Ratio-10 %" rows): the average budget
                              per head follows the context, floor(r * tokens) kept within [max(1, min_budget),
                              budget_per_head]; set uniformly when the prompt is loaded and used as Algorithm 2's
                              B_total (times L * H) at every reallocation.  budget_per_head still sizes the
                              storage.  0 = fixed budgets */
} crystalkv_config_t;

/*
 * Allocates the handle's device state (pool, lists, metadata, lambda^D table, split-K
 * scratch).  Section 5: one cache per (layer, head) with CRF and tau per entry.
 * Errors: EINVAL (bad field, *out untouched), ENOMEM, ECUDA.
 */
int crystalkv_create(const crystalkv_config_t* cfg, crystalkv_t** out);

/* Frees everything the handle owns.  NULL is accepted. */
int crystalkv_destroy(crystalkv_t* h);

/*
 * Loads a prompt into one layer (Algorithm 1 inputs K/V, Q^last) and runs one
 * Algorithm 1 pass with Q^last at t = P-1, so CRF/tau are seeded and heads whose
 * prompt exceeds their budget are evicted down to it.
 *   k, v   dev  [batch][P][H][128]     q_last dev [batch][Hq][128] (query of token P-1)
 * A prompt longer than the budget is scored from k and q_last as they are, and only the rows
 * of the entries Algorithm 1 retains are stored, so the pool never holds more than the budget.
 * P must satisfy 1 <= P < max_context and P <= max_budget + evict_every + max_answer_tokens (the
 * heads' list capacity).  Errors: EINVAL; ESTATE if the layer was prefilled.
 */
int crystalkv_prefill(crystalkv_t* h, int layer, const void* k, const void* v,
                      const void* q_last, int P, void* stream);

/*
 * Loads a prompt into one layer and replays Algorithm 1 over an observation window: the
 * queries of the last W prompt tokens, in order.  Token i arrives with CRF 0 and tau = i;
 * the query of token t (P-W <= t <= P-1) attends to tokens 0..t (causal) and runs steps 1-3
 * at time t; step 4 runs once, after the last query, and brings every head down to its budget.
 * W = 1 retains what crystalkv_prefill retains (tau of never-hit entries is their position
 * instead of P-1).
 *   k, v       dev [batch][P][H][128]
 *   q_window   dev [W][batch][Hq][128]   queries of tokens P-W .. P-1
 *   out_window dev [W][batch][Hq][128]   their attention outputs, or NULL
 * All buffers belong to the caller and must stay valid until the work queued on `stream`
 * has run.  1 <= W <= P, and P <= budget_per_head + max_answer_tokens in evict mode (the window's
 * outputs need every token's values, so the whole prompt is stored before the one eviction).
 * FullKV mode: only the insertion
 * (and out_window, if asked for, stays untouched).  Errors: EINVAL; ESTATE if the layer was prefilled.
 */
int crystalkv_prefill_window(crystalkv_t* h, int layer, const void* k, const void* v,
                             const void* q_window, int P, int W, void* out_window, void* stream);

/*
 * One decode step of one layer for all sequences (Section 2.2 attention fused with
 * Algorithm 1): appends (k_new, v_new) at time t = previous t + 1, attends the G
 * queries of every kv head over its cache, writes `out`, and in the think stage of
 * evict mode marks the top-p hit entries, updates CRF/tau (steps 2-3) and evicts the
 * lowest-CRF entry of every head that is over budget (step 4); the next arriving token
 * takes its place.
 *   q, out dev [batch][Hq][128]        k_new, v_new dev [batch][H][128]
 * Errors: EINVAL; ESTATE before prefill or when t would reach max_context or a head
 * would outgrow its capacity.
 */
int crystalkv_decode_step(crystalkv_t* h, int layer, const void* q, const void* k_new,
                          const void* v_new, void* out, void* stream);

/*
 * The same step with HOST buffers (page-locked for asynchronous copies; pageable memory works
 * but its copies block the host).  The inputs are brought up on one stream of the handle (by
 * one small kernel that reads the page-locked buffers through their device mapping, else by
 * three copies) and `out` is copied down on another, both ordered
 * against the step on `stream` by events, so the copies of one layer run beside the kernels
 * of others.  No host synchronisation.  `out_host` is complete once `stream` has passed a
 * later crystalkv_join (or any call that reads the cache state) and has been synchronised;
 * the input buffers may be reused from then on too.
 */
int crystalkv_decode_step_host(crystalkv_t* h, int layer, const void* q_host,
                               const void* k_new_host, const void* v_new_host, void* out_host,
                               void* stream);

/*
 * Makes `stream` wait (on the device, without blocking the host) for all work the handle
 * has enqueued on its internal stream: the Algorithm 1 kernels of earlier decode steps,
 * which run behind the attention kernels so that they overlap the next layer.  `out` of
 * a decode step never needs this; every call that reads or edits the cache state does it
 * by itself.  Use it before recording an event that should cover whole steps.
 */
int crystalkv_join(crystalkv_t* h, void* stream);

/* Section 4 splits a generation into the think stage, whose cache is compressed, and the
 * answer stage.  Think stage: Algorithm 1 runs.  Answer stage: the think cache is frozen, new
 * tokens are appended beyond the budget and attended, nothing is tracked or evicted. */
int crystalkv_set_stage(crystalkv_t* h, int stage);

/*
 * Algorithm 2 (Section 5.3), per sequence: aggregates every head's CRF decayed to the
 * time of the last step, recomputes integer budgets that sum to B_total, and makes
 * heads whose budget shrank evict down to it; the pages they no longer need return to the
 * sequence's free list for heads that grew.  All layers must be at the same time step.
 * Errors: ESTATE (layers out of step, FullKV mode, before prefill).
 */
int crystalkv_rebudget(crystalkv_t* h, void* stream);

/*
 * Algorithm 1's output `Retain` as token positions: those kept by (layer, seq, kv_head),
 * ascending, into host memory.  Synchronises `stream`.  *n_out receives the count; ESTATE if
 * cap is too small.
 */
int crystalkv_get_retained(crystalkv_t* h, int layer, int seq, int kv_head,
                           int32_t* pos_out_host, int32_t cap, int32_t* n_out, void* stream);

/* Algorithm 2's output B': the current budgets, host int32 [batch][L][H].  Synchronises `stream`. */
int crystalkv_get_budgets(crystalkv_t* h, int32_t* out_host, void* stream);

/*
 * The state Algorithm 1 keeps per entry of one head (its inputs CRF and tau, next to the
 * entry's token position), sorted by position: records of three int32 {position, CRF as fp32
 * bits, tau}.  host_buf holds cap records; *n receives the count.  Synchronises `stream`.
 */
int crystalkv_export_state(crystalkv_t* h, int layer, int seq, int kv_head, int32_t* host_buf,
                           int32_t cap, int32_t* n, void* stream);

/*
 * The other two inputs of Algorithm 1, K and V, of one head: its entries' rows in the order
 * of crystalkv_export_state's records, host bf16 [n][128] each (cap rows of room).  *n
 * receives the count.  Synchronises `stream`.
 */
int crystalkv_export_kv(crystalkv_t* h, int layer, int seq, int kv_head, void* k_rows_host,
                        void* v_rows_host, int32_t cap, int32_t* n, void* stream);

/*
 * The inverse of the two exports: replaces the content of one head by n entries given as
 * records {position, CRF bits, tau} (any order) with their K and V rows, host bf16 [n][128]
 * each, and sets the head's budget (Algorithm 1's input B; 0 keeps the current one) and the
 * layer's time t (the time of its last completed step, Algorithm 1's input t).  The head returns
 * the pool pages it no longer needs and takes those it lacks.  A layer that was never
 * prefilled becomes usable once every one of its heads has been imported with the same t: a
 * handle can be rebuilt from the exports of another (with crystalkv_set_stage for the stage).
 * Synchronises `stream`.  Errors: EINVAL (n outside [1, list capacity), budget outside
 * [0, max_budget], a position or tau after t), ESTATE (the layer is at another time), ECHECK
 * later from crystalkv_check if the sequence's pool had no pages left.
 */
int crystalkv_import_state(crystalkv_t* h, int layer, int seq, int kv_head,
                           const int32_t* host_buf, int32_t n, const void* k_rows_host,
                           const void* v_rows_host, int32_t budget, int32_t t, void* stream);

/* Sets one head's budget (Algorithm 1's input B) directly; a head holding more evicts down to
 * it at once, as after a reallocation. */
int crystalkv_set_budget(crystalkv_t* h, int layer, int seq, int kv_head, int32_t budget,
                         void* stream);

/* Time step of the layer's last completed step (P-1 after prefill, -1 before). */
int crystalkv_time(crystalkv_t* h, int layer);

/*
 * Bytes the Section 2.2 / Algorithm 1 data flow must move for the steps run so far:
 * *kv_bytes = sum over steps and heads of entries attended * 512 (K and V rows).
 * Synchronises `stream`; counters are kept on the device and cost one atomic per head.
 */
int crystalkv_get_counters(crystalkv_t* h, uint64_t* entries_attended, uint64_t* hits,
                           uint64_t* evictions, void* stream);

/* Reads and clears the handle's device error word (0 = clean).  Synchronises `stream`. */
int crystalkv_check(crystalkv_t* h, void* stream);

/*
 * Debug check of page ownership (the in-place reuse of Algorithm 1 step 4 and the hand-over
 * of pool pages between heads by the reallocation): every pool page (16 entries) of every
 * sequence must be held exactly once, by the sequence's free list or by one head, and every
 * head must hold the pages that back its entries and the place of its next arrival.
 * Allocates a temporary, synchronises `stream`; not for the hot path.  ECHECK on failure,
 * ESTATE before every layer is prefilled.
 */
int crystalkv_validate(crystalkv_t* h, void* stream);

/*
 * crystalkv_validate for callers that must not allocate device memory.  (The paper has no
 * counterpart: this is a service of the library, like crystalkv_validate itself.)
 *
 * crystalkv_validate takes a temporary from cudaMalloc on every call.  That is not possible
 * where a framework has already claimed all device memory for its own pool (cudaMalloc then
 * fails although the framework has room), or in a serving loop that may not take the
 * device-wide synchronisation a cudaMalloc / cudaFree pair implies.  This entry point does the
 * same check with its per-page counters in an array that is built into the library: it calls
 * no cudaMalloc, cudaFree or other allocating routine.  Like crystalkv_validate it copies its
 * verdict to the host and synchronises `stream`.
 *
 *   counts_out_host  host int32[2] or NULL: [0] page ids or counts out of range, [1] pages not
 *                    owned exactly once (both 0 on a sound handle)
 *
 * Limits and rules
 *   - The array covers handles of at most 2^17 = 131 072 pool pages in total (1 GiB of K/V
 *     rows).  A handle has batch * (ceil(L * H * E / 16) + L * H) pages, with E = budget_per_head
 *     + evict_every + max_answer_tokens + 1 entries per head in evict mode and max_context + 1
 *     in FullKV mode.  A larger handle is refused with EINVAL and a message that says so; use
 *     crystalkv_validate there.
 *   - Every GPU on which the library is loaded holds the array (512 KiB) until the process ends.
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress,
 *     with that device made current); later calls on that device reuse it.
 *   - All calls on one GPU, from any handle, share the array, and it keeps the previous
 *     call's contents; each call clears the part it uses on `stream` first.  Two calls whose
 *     work overlaps on the GPU (different streams, no ordering between them) race: order them.
 *   - Like crystalkv_validate it synchronises `stream` and is not for the hot path.
 * Errors: EINVAL (NULL handle, too many pages, device ordinal above 63), ESTATE before every
 * layer is prefilled, ECUDA, ECHECK when ownership is broken.
 */
int crystalkv_validate_static(crystalkv_t* h, int32_t* counts_out_host, void* stream);

/*
 * Test hook for the two ownership checks (the paper has no counterpart): overwrites entry
 * `index` of one head's page table with `page`, both checked against their ranges (EINVAL).
 * A handle treated this way is inconsistent on purpose: it may be validated and destroyed,
 * nothing else.  Synchronises `stream`.
 */
int crystalkv_debug_set_page(crystalkv_t* h, int layer, int seq, int kv_head, int32_t index,
                             int32_t page, void* stream);

/*
 * Test hook (the paper has no counterpart): copies the launch plan of a layer's next attention
 * kernel to the host.  hdr_host[4] = {pieces, groups (pages of 16 keys) over all heads, warps the
 * plan is made for, 1 when it is for a decode step}; wrange_host[2 w], [2 w + 1] = the pieces
 * [first, end) that warp w of the grid (CTA w / 8) streams, for w < hdr[2]; desc_host[4 i ..] =
 * {head index seq * n_kv_heads + kv_head, j, k, together} of piece i: the j-th of the head's k
 * pieces, `together` = 1 when the k pieces sit in consecutive warps of one CTA, 2 when they sit
 * that way in runs of eight (pieces 8 r .. 8 r + 7 in the eight warps of one CTA) and one shorter
 * run, 0 otherwise.  warps_cap and pieces_cap are the capacities of the two arrays in warps and
 * in pieces; EINVAL unless warps_cap >= 8 x SMs and pieces_cap >= 8 x SMs + batch x n_kv_heads.
 * Synchronises `stream`.
 */
int crystalkv_debug_get_plan(crystalkv_t* h, int layer, int32_t* hdr_host, int32_t* wrange_host,
                             int32_t warps_cap, int32_t* desc_host, int32_t pieces_cap, void* stream);

/*
 * Test hook for the launch planner's counting rule (the paper has no counterpart; needs no GPU
 * and no handle): the number of CTAs of eight warps that hold `whole_ctas` CTAs taken whole plus
 * runs_by_length[s] runs of s consecutive warps, s = 1 .. 7 (entry 0 is ignored; host int32[8]),
 * when the runs are placed longest first, each into the open CTA with the fewest free warps that
 * still holds it.  Returns that count (>= 0), or EINVAL for a NULL array or a negative entry.
 */
int crystalkv_debug_ctas_needed(int32_t whole_ctas, const int32_t* runs_by_length);

const char* crystalkv_strerror(int code);
const char* crystalkv_last_error(crystalkv_t* h);

#ifdef __cplusplus
}
#endif
#endif /* CRYSTALKV_H */
