/* tide.h — C ABI of the tide-kv library (B200 / sm_100a only).
 *
 * The GPU hot path behind Continuous Task Batching (CTB, paper Section 4):
 * rollout tasks that pause for an external environment keep their KV state
 * resident and resume with the observation tokens appended, instead of
 * re-running prefill over their history (paper Section 1, first challenge;
 * Section 2.2).  Per engine step the GPU work is (a) appending each task's
 * new K/V rows into a paged cache and (b) grouped-query attention of a mixed
 * batch — one-token decode rows next to multi-token resume rows whose causal
 * queries see the whole preserved prefix.
 *
 * Conventions
 *   - One tide_kv_t per GPU (a rollout data-parallel rank is its own token
 *     budget pool with its own cache, Section 4.1).  One caller thread per
 *     tide_kv_t.  The CUDA device current at tide_kv_create must be current
 *     at every later call.
 *   - "host" pointers are ordinary host memory read during the call; "device"
 *     pointers are device memory on that GPU, 16-byte aligned, owned by the
 *     caller and never freed or reallocated by the library.
 *   - Device work is enqueued on `stream` (a cudaStream_t passed as void*);
 *     host bookkeeping is updated before the call returns.  append followed by
 *     attend on one stream is ordered.
 *   - Every call returns TIDE_OK (0) or a negative tide_status_t.  All
 *     validation happens before any mutation: a failing call changes nothing.
 *     There is no CPU fallback anywhere.
 *   - Values are bf16 (raw 16-bit patterns); accumulation is fp32.
 */
#ifndef TIDE_H_
#define TIDE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  TIDE_OK = 0,
  TIDE_ERR_INVALID_ARG = -1,    /* NULL / misaligned pointer, bad geometry, bad indptr, bad layer      */
  TIDE_ERR_UNKNOWN_TASK = -2,   /* task id not registered by tide_kv_alloc                             */
  TIDE_ERR_TASK_EXISTS = -3,    /* tide_kv_alloc of a live task                                        */
  TIDE_ERR_DUPLICATE_TASK = -4, /* the same task twice in one tide_kv_append                           */
  TIDE_ERR_NO_PAGES = -5,       /* free pages cannot hold the request (the caller pauses or evicts,    */
                                /* Algorithm 1, eviction loop)                                         */
  TIDE_ERR_TABLE_FULL = -6,     /* a task would exceed max_pages_per_task                              */
  TIDE_ERR_CTX_RANGE = -7,      /* a row violates 1 <= q_len <= ctx_len <= resident length             */
  TIDE_ERR_WORKSPACE = -8,      /* pool / workspace / batch limits too small for the request           */
  TIDE_ERR_CUDA = -9,           /* a CUDA runtime call failed                                          */
  TIDE_ERR_DEVICE_TIMEOUT = -10 /* a bounded wait inside a kernel ran out (reported by tide_status)    */
} tide_status_t;

typedef struct tide_kv tide_kv_t; /* opaque */

/* One batch row of tide_attend.  ctx_len is the number of cached tokens the row
 * attends over INCLUDING this step's q_len appended tokens; the preserved
 * prefix is ctx_len - q_len.  A decode row has q_len 1. */
typedef struct {
  int32_t task;
  int32_t q_len;
  int32_t ctx_len;
} tide_row_t;

typedef struct {
  int32_t num_layers;         /* L in [1, 256]: K/V stores that share one page table (layer l of a   */
                              /* model); the pool holds L * num_pages pages                         */
  int32_t num_q_heads;        /* Hq, a multiple of num_kv_heads, Hq/Hkv <= 16                       */
  int32_t num_kv_heads;       /* Hkv                                                                */
  int32_t head_dim;           /* D: 64 or 128                                                       */
  int32_t page_size;          /* S: 16 or 32 tokens                                                 */
  int32_t max_tasks;          /* task ids are dense ints in [0, max_tasks)                          */
  int32_t max_pages_per_task; /* page-table row length                                              */
  int32_t max_batch_rows;     /* most rows / tasks in one tide_attend / tide_kv_append              */
  int64_t num_pages;          /* pool capacity in pages                                             */
  int64_t max_batch_tokens;   /* most query tokens in one tide_attend (sum of q_len) and most new   */
                              /* tokens in one host-buffer step                                     */
  void* pool;                 /* device; >= pool_bytes from tide_kv_required_bytes, 1024-B aligned  */
  size_t pool_bytes;
  void* workspace;            /* device scratch; >= workspace_bytes, 256-B aligned                  */
  size_t workspace_bytes;
  const int32_t* free_order;  /* host; permutation of [0, num_pages): the order in which a fresh    */
                              /* pool hands pages out.  NULL = identity.                            */
} tide_kv_config_t;

/* Sizes the caller must provide for cfg's geometry (pool / workspace fields of cfg are ignored). */
int tide_kv_required_bytes(const tide_kv_config_t* cfg, size_t* pool_bytes, size_t* workspace_bytes);

/* Creates the cache object: host bookkeeping, a pinned staging ring, device tables carved from
 * cfg->workspace.  The pool is NOT cleared.  Physical page layout inside the pool is private to the
 * library; read logical content back with tide_kv_read. */
int tide_kv_create(const tide_kv_config_t* cfg, tide_kv_t** out);
int tide_kv_destroy(tide_kv_t* kv);

/* Flush every task and restart the free stack from free_order (NULL = identity): the cache flush
 * that follows each weight synchronisation (Section 5.2, rollout shrink / KV-cache reset). */
int tide_kv_reset(tide_kv_t* kv, const int32_t* free_order);

/* Register `task` with length 0 (Section 4.1, token-aware admission).  Takes no pages; pages are
 * taken by tide_kv_append.  reserve_tokens is an admission check only: the call fails with
 * TIDE_ERR_NO_PAGES unless free_pages * page_size >= reserve_tokens (0 = no check). */
int tide_kv_alloc(tide_kv_t* kv, int32_t task, int64_t reserve_tokens);

/* Append indptr[j+1]-indptr[j] tokens to task_ids[j] for j in [0, n_tasks) (the resume step of
 * Section 4: observation tokens are added to the preserved state).  new_k / new_v: device bf16
 * [T, Hkv, D], T = indptr[n_tasks], token rows of task j at [indptr[j], indptr[j+1]).
 * Pages are popped from the free stack in array order, one each time a token lands on slot 0 of a
 * new logical page.  All-or-nothing: on any error no task changes.  Zero-length entries are no-ops. */
int tide_kv_append(tide_kv_t* kv, int32_t layer, int32_t n_tasks, const int32_t* task_ids /*host*/,
                   const int32_t* indptr /*host, n_tasks+1*/, const void* new_k /*device*/,
                   const void* new_v /*device*/, void* stream);

/* A model with L layers keeps L K/V stores that grow in lock step: one page table and one set of lengths serve
 * all of them (the paper's token budget of Section 4.1 counts tokens, not layers).  With num_layers > 1 an
 * append is therefore split: tide_kv_extend grows the tasks once per step (pages, lengths, the device page
 * table, and on every layer the private copy of a shared partial page) and writes no K/V;
 * tide_kv_write(layer) then puts that layer's new rows into the LAST indptr[j+1]-indptr[j] positions of
 * task_ids[j] (TIDE_ERR_CTX_RANGE if a task is shorter than that).  tide_kv_append is tide_kv_extend followed by
 * tide_kv_write on layer 0, and accepts layer 0 only.  Argument meaning, all-or-nothing behaviour and errors
 * are those of tide_kv_append. */
int tide_kv_extend(tide_kv_t* kv, int32_t n_tasks, const int32_t* task_ids /*host*/,
                   const int32_t* indptr /*host, n_tasks+1*/, void* stream);
int tide_kv_write(tide_kv_t* kv, int32_t layer, int32_t n_tasks, const int32_t* task_ids /*host*/,
                  const int32_t* indptr /*host, n_tasks+1*/, const void* new_k /*device*/,
                  const void* new_v /*device*/, void* stream);

/* Attention of a mixed continuous batch over the cache (Section 3.2: concurrent multi-task
 * generation on one rank; Section 4: resumed tasks continue from preserved state).
 * Row b: query i in [0, q_len) sits at position ctx_len - q_len + i and sees keys [0, that position]
 * (causal inside the appended chunk, full attention to the preserved prefix).  Query head h reads KV
 * head h / (Hq/Hkv).  q, out: device bf16 [sum q_len, Hq, D], rows concatenated in batch order;
 * lse: device fp32 [sum q_len, Hq] (natural log of the sum of exp of scaled logits) or NULL.
 * page_table: device int32 [max_tasks][max_pages_per_task] to read instead of the library's own
 * table, or NULL.  The same task may appear in several rows.  Read-only on the cache. */
int tide_attend(tide_kv_t* kv, int32_t layer, int32_t n_rows, const tide_row_t* rows /*host*/,
                const int32_t* page_table /*device or NULL*/, const void* q /*device*/, float scale,
                void* out /*device*/, float* lse /*device or NULL*/, void* stream);

/* One whole CTB step from HOST buffers: copies new_k / new_v / q to the device, appends q_len
 * tokens to every row's task (rows must name distinct tasks; ctx_len must equal the resident length
 * after the append), attends, and copies out / lse back.  new_k, new_v: host bf16 [sum q_len, Hkv, D];
 * q, out: host bf16 [sum q_len, Hq, D]; lse: host fp32 or NULL.  Host buffers should be pinned for
 * the copies to be asynchronous.  The call returns after the results have arrived.  A small step (up to
 * 2 MiB in all) whose buffers are pinned and addressable by the device is not copied at all: the kernels
 * read the inputs and write the results across PCIe themselves.  A large step is cut
 * into groups of consecutive rows whose copies (on two streams the library owns) run beside the kernels
 * of other groups; pages, cache contents and results do not depend on the cut.  The whole step is checked
 * (rows, duplicates, pages) before anything is copied or changed.  Takes layer 0 only. */
int tide_step_host(tide_kv_t* kv, int32_t layer, int32_t n_rows, const tide_row_t* rows /*host*/,
                   const void* new_k /*host*/, const void* new_v /*host*/, const void* q /*host*/,
                   float scale, void* out /*host*/, float* lse /*host or NULL*/, void* stream);

/* One CTB step of a model with several layers, planned once.  tide_step_begin takes the step's rows (distinct
 * tasks; ctx_len must equal the resident length after q_len tokens are added, as in tide_step_host), grows the
 * tasks (tide_kv_extend), plans the attention work and uploads the plan and the write records to a part of the
 * workspace that stays valid until the next tide_step_begin or any call that changes a task.  All-or-nothing.
 * tide_step_layer(layer) then writes that layer's new_k / new_v (device bf16 [sum q_len, Hkv, D], batch order)
 * and attends q against layer `layer` exactly as tide_attend would; it only launches kernels (no copies, no
 * events, no host waits), so the calls of all layers may be captured in one CUDA graph and replayed, as long
 * as the captured pointers stay valid.  scale must be positive and finite.  TIDE_ERR_INVALID_ARG if no step is
 * open.  Per-phase timing (tide_set_profiling) does not cover tide_step_layer. */
int tide_step_begin(tide_kv_t* kv, int32_t n_rows, const tide_row_t* rows /*host*/, void* stream);
/* Fixes the launch shapes of tide_step_layer so that ONE captured CUDA graph of a step's layers can be replayed
 * for later steps with other rows: every kernel is launched with a grid sized for the given maxima (work items of
 * the decode-style, warp-MMA tile and tcgen05 kernels, rows of the merge, new tokens) and reads the step's real
 * counts from the step area that tide_step_begin fills; surplus thread blocks leave at once.  A maximum of 0
 * means that kind of launch is left out.  tide_step_begin refuses a step that plans more than a maximum with
 * TIDE_ERR_WORKSPACE (tide_last_plan shows what a step planned).  All five 0 turns the mode off (the default:
 * exact grids).  Closes an open step.  max_tokens may not exceed max_batch_tokens. */
int tide_step_fix_grids(tide_kv_t* kv, int32_t max_decode_items, int32_t max_tile_items, int32_t max_umma_items,
                        int32_t max_merge_rows, int32_t max_tokens);
int tide_step_layer(tide_kv_t* kv, int32_t layer, const void* new_k /*device*/, const void* new_v /*device*/,
                    const void* q /*device*/, float scale, void* out /*device*/, float* lse /*device or NULL*/,
                    void* stream);

/* Return the task's pages to the free stack, last page first, and forget the task (task end or
 * eviction, Algorithm 1).  Host only; page contents are not cleared. */
int tide_kv_release(tide_kv_t* kv, int32_t task);

/* Roll a live task back to new_len <= its length, returning pages ceil(new_len/S).. last-to-first
 * (sliding-window pruning of old observations, Appendix C.2).  Host only. */
int tide_kv_truncate(tide_kv_t* kv, int32_t task, int32_t new_len);

/* Group-shared prefixes (a GRPO group rolls out G trajectories from one prompt, Section 2.1; CTB's worker
 * affinity keeps a group on the rank that holds its shared prefix, end of Section 4).  `child` becomes a live
 * task whose content is the parent's current content: the parent's full pages are SHARED (reference counted,
 * never written again), a partial last page is copied into a fresh page, so parent and child can both keep
 * appending.  A page returns to the free stack when its last holder lets go of it.  An append that would write
 * into a page other tasks still hold (possible after tide_kv_truncate into shared pages) first replaces it by
 * a private copy, taken from the free stack before the task's other new pages.  Page copies cover every
 * layer; `layer` must be 0.  Errors: TIDE_ERR_TASK_EXISTS, TIDE_ERR_UNKNOWN_TASK, TIDE_ERR_NO_PAGES (no page
 * for the copy). */
int tide_kv_fork(tide_kv_t* kv, int32_t layer, int32_t parent, int32_t child, void* stream);
/* How many tasks hold each page of `task` (same order as tide_kv_page_table). */
int tide_kv_page_refs(tide_kv_t* kv, int32_t task, int32_t* out /*host*/, int32_t cap, int32_t* n_pages);

/* tide_kv_release for several tasks at once (a finished GRPO group, or every task a scheduler evicts in one
 * pass of Algorithm 1).  All-or-nothing: unknown or repeated ids release nothing. */
int tide_kv_release_many(tide_kv_t* kv, int32_t n_tasks, const int32_t* task_ids /*host*/);

/* Sliding-window pruning of old observations (Appendix C.2: only the most recent images are kept, which splits
 * the trajectory): the task keeps tokens [0, keep_prefix) and [tail_begin, len); the tokens in between are
 * dropped and the tail moves down to start at keep_prefix.  Equivalent, page table included, to reading the
 * tail, tide_kv_truncate(task, keep_prefix) and appending the tail again; the move runs on `stream` through
 * the workspace staging area and covers every layer (`layer` must be 0).  Requires
 * 0 <= keep_prefix <= tail_begin <= len.  All-or-nothing: TIDE_ERR_NO_PAGES if the shorter task could not get
 * its pages (only possible when it shares pages, which do not come back to the free stack);
 * TIDE_ERR_WORKSPACE if the task shares a page from position keep_prefix on and its tail is longer than
 * max_batch_tokens (such a tail has to be staged whole). */
int tide_kv_prune(tide_kv_t* kv, int32_t layer, int32_t task, int32_t keep_prefix, int32_t tail_begin, void* stream);

/* Introspection (the per-rank token usage CTB schedules on, Section 4.1 / Algorithm 1). */
int tide_kv_task_len(tide_kv_t* kv, int32_t task, int32_t* len);
int tide_kv_page_table(tide_kv_t* kv, int32_t task, int32_t* out /*host*/, int32_t cap, int32_t* n_pages);
int tide_kv_usage(tide_kv_t* kv, int64_t* used_tokens, int64_t* free_pages);
/* Logical content of a task as contiguous device bf16 [len, Hkv, D] (out_k / out_v). */
int tide_kv_read(tide_kv_t* kv, int32_t layer, int32_t task, void* out_k /*device*/, void* out_v /*device*/,
                 void* stream);

/* Synchronises `stream` and returns the device status word: TIDE_OK, or TIDE_ERR_DEVICE_TIMEOUT if a
 * bounded wait in a kernel ran out since the last call (the word is then cleared).  Every wait inside the
 * attention kernels (for a K/V stage, a tensor-core result, a free buffer) has a time limit; when one runs out
 * the thread block records the time-out, finishes without waiting again and frees what it holds, and the kernel
 * returns by itself.  The word is sticky: from the time-out until this call clears it, thread blocks of that
 * launch and of every later attention launch on the handle leave without computing, so `out` / `lse` of those
 * calls are undefined although the calls themselves returned TIDE_OK.  A caller that needs to know asks
 * tide_status after the step; after a TIDE_ERR_DEVICE_TIMEOUT the cache contents are intact and the attention
 * call can simply be repeated. */
int tide_status(tide_kv_t* kv, void* stream);

/* Rows of the most recently planned batch (tide_attend, tide_step_begin) that were planned as groups sharing their
 * first pages: consecutive decode rows of distinct tasks whose page tables agree on at least 256 tokens of full
 * pages (tasks made by tide_kv_fork).  The shared pages of a group are then read once for all its rows - the
 * group's queries form one multi-query work item over them - and each row's own pages once, the two parts being
 * combined by the same log-sum-exp merge that combines KV splits.  Results are those of tide_attend row by row
 * (same tolerance); no grouping when the caller supplies its own page table. */
int tide_last_sharing(tide_kv_t* kv, int64_t* groups, int64_t* rows);

/* Counters of the most recent tide_attend: work items launched on the decode-style and the
 * tensor-tile paths, rows merged, and kernels launched by the most recent append + attend pair. */
int tide_last_plan(tide_kv_t* kv, int64_t* decode_items, int64_t* prefill_items, int64_t* merge_rows,
                   int64_t* kernel_launches);

/* Planner settings and test hooks of one handle.  The defaults are the measured best on B200; nothing reads the
 * environment.  Changing a setting closes an open step (tide_step_begin must be called again).
 * TIDE_ERR_INVALID_ARG for an unknown knob or a value outside its range. */
typedef enum {
  TIDE_TUNE_ITEMS_PER_SM = 0,     /* work items per SM the KV-split planner aims for, 1..64 (default 3)            */
  TIDE_TUNE_GROUPING = 1,         /* 0: never plan forked rows as groups that read shared pages once (default 1)   */
  TIDE_TUNE_MIN_SAVED_BYTES = 2,  /* KV bytes a batch must save before groups are used (default 64 MiB)            */
  TIDE_TUNE_HOST_STEP_CHUNKS = 3, /* row groups of tide_step_host, 1..8; 0 = chosen by transfer size (default)     */
  TIDE_TUNE_UMMA_MIN_ROWS = 4,    /* packed rows (q_len * Hq/Hkv) from which a head_dim-128 row runs on the        */
                                  /* tcgen05 kernel, >= 17 (default 17)                                            */
  TIDE_TUNE_WAIT_LIMIT_US = 5,    /* time limit of every wait inside a kernel, microseconds (default 2 000 000)    */
  TIDE_TUNE_UMMA_TILE_KEYS = 7,   /* key-tile size of the tcgen05 kernel: 64 or 128                                */
  TIDE_TUNE_UPLOAD_BY_KERNEL = 8, /* the small planning uploads of every call are done by a kernel that reads the   */
                                  /* pinned, device-mapped staging slot (default 1) or by the copy engine (0)       */
  TIDE_TUNE_INLINE_DESCRIPTORS = 9, /* small appends (<= 128 rows, <= 256 new pages) and decode-only batches of up  */
                                  /* to 128 rows carry their descriptors in the launch's own parameters, so that  */
                                  /* nothing is uploaded before the kernel (default 1); 0: always upload           */
  TIDE_TUNE_HOST_ZERO_COPY = 10,  /* tide_step_host: a step of up to 2 MiB whose host buffers are pinned and mapped   */
                                  /* is not copied; the kernels read and write the host buffers themselves         */
                                  /* (default 1); 0: always copy                                                  */
  TIDE_TUNE_DROP_FIRST_STAGE = 6  /* test hook, non-zero arms it for the NEXT attention call only: in work item 0   */
                                  /* of each attention kernel of that call the K/V producer leaves out (its part   */
                                  /* of) the first stage, so the wait for that stage runs out and the time-out     */
                                  /* path of tide_status can be exercised without any fault.  Results of that      */
                                  /* call are undefined.                                                           */
} tide_tune_t;
int tide_tune(tide_kv_t* kv, int knob, int64_t value);

/* Per-phase device timing of the calls that follow (CUDA events on the caller's stream; off by default).
 * tide_phase_ms waits for the most recent tide_attend and returns the milliseconds spent in the most
 * recent tide_kv_append (0 if none since the last query), in the decode-style attention kernel, in the
 * tensor-tile attention kernel and in the merge kernel: the split of one mixed CTB step into its
 * KV-bandwidth-bound and its tensor-bound halves. */
int tide_set_profiling(tide_kv_t* kv, int enable);
int tide_phase_ms(tide_kv_t* kv, float* append_ms, float* decode_ms, float* tile_ms, float* merge_ms);

/* (The paper has no counterpart to this call; it exists for callers of this library.)
 * Attention for decode-style rows (q_len * Hq/Hkv <= 16) that allocates nothing, neither on the device nor on
 * the host.  tide_attend parks the partial results of its KV splits and its row descriptors in the workspace
 * that the caller allocated; this variant keeps both in a fixed array compiled into the library (about 8 MB of
 * device memory on every GPU that loads the library, held until the process exits).  It is meant for callers
 * that cannot allocate at the time they need attention: code running while a CUDA graph is being captured in
 * global mode, where cudaMalloc is refused; processes whose framework allocator already owns the whole device,
 * so a fresh cudaMalloc fails; and steps that cannot afford the device-wide synchronisation cudaMalloc implies.
 * Same semantics, arguments and results as tide_attend restricted to such rows, with the library's own page
 * table, on layer 0.  Limits: at most TIDE_STATIC_MAX_ROWS rows per call (more returns TIDE_ERR_WORKSPACE), decode-style
 * rows only (others return TIDE_ERR_INVALID_ARG); long rows are split over KV only as far as the fixed array
 * allows.  The first call on a device looks up the array's device address; make that call before any stream
 * capture begins.  The device the handle was created on must be current (TIDE_ERR_INVALID_ARG otherwise).  The
 * call copies nothing from host memory: the row records travel as kernel arguments and are expanded on the
 * device, so it is asynchronous on `stream`.  Every call uses the same array and overwrites what the previous
 * call left there (every record a call reads it has written itself, so nothing needs clearing between calls),
 * and two calls whose kernels may overlap on the GPU (different streams) race: keep the calls of one process on
 * one stream, or order them with events. */
#define TIDE_STATIC_MAX_ROWS 64
int tide_attend_decode_static(tide_kv_t* kv, int32_t n_rows, const tide_row_t* rows /*host*/,
                              const void* q /*device*/, float scale, void* out /*device*/,
                              float* lse /*device or NULL*/, void* stream);

const char* tide_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* TIDE_H_ */
