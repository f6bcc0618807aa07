/*
 * lazyev -- LazyEviction decode / track / evict hot path for NVIDIA B200 (sm_100a).
 *
 * One handle serves `units = layers * batch * kv_heads` independent cache units;
 * unit u = (layer * batch + b) * kv_heads + h.  Every unit holds the same number
 * of cached tokens n (all sequences were prefilled with the same length and are
 * decoded in lock step), at most `capacity = max(budget, max_prefill) + window`.
 *
 * Conventions
 *   - Every call returns 0 (LAZYEV_OK) or a negative LAZYEV_E* code; nothing
 *     throws or aborts.  lazyev_last_error() gives the message of the last
 *     failure on a handle, lazyev_strerror() names a code.
 *   - "device pointer" arguments are contiguous arrays in the memory of the GPU
 *     that was current at lazyev_bind(); activations are bfloat16 (raw 16-bit
 *     patterns), head_dim = 128 elements per row.
 *   - The caller owns all device memory and the CUDA stream.  The library
 *     allocates no device memory at all; it owns only the host-side handle and a
 *     few internal CUDA streams and events (a low-priority stream for the second
 *     decode launch of a step, two copy streams for the host-buffer entry point),
 *     created on first use and destroyed with the handle; their work is always
 *     joined into the bound stream before a call returns control to it.
 *   - Calls are asynchronous on the bound stream unless stated otherwise.
 *     A handle must not be used from two threads at once.
 *
 * Device memory layout (described so that callers can size and inspect it)
 *   kv_pool : pages of 64 tokens; one page = 64 K rows (256 B each) followed by
 *             64 V rows.  Inside a row the eight-element (16-byte) chunk c of
 *             token slot r is stored at chunk position c ^ (r & 7) (low three
 *             bits), which makes a linear bulk copy of a page land in shared
 *             memory free of ldmatrix bank conflicts.  Slot i of unit u lives
 *             in physical page page_table[u][i / 64], row i % 64.
 *   state   : page table, and per unit and slot: the pair (TS, MRI) as two int32 side by side,
 *             original position (int32), last probability (float32).
 *   scratch : eviction source lists, staging for the host-buffer entry point, score
 *             staging for lazyev_dump_state, the MRI histogram.
 */
#ifndef LAZYEV_H
#define LAZYEV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lazyev lazyev_t;

enum {
    LAZYEV_OK = 0,
    LAZYEV_EINVAL = -1,    /* bad argument (null pointer, unsupported shape, out-of-range value) */
    LAZYEV_ESTATE = -2,    /* call made in the wrong state (e.g. decode before prefill)           */
    LAZYEV_ECAPACITY = -3, /* the cache of a unit would grow past its capacity                    */
    LAZYEV_EDEVICE = -4,   /* a kernel reported a failure in the device status word                */
    LAZYEV_ECUDA = -5      /* a CUDA runtime call failed                                           */
};

/* Importance score variants: Eq. (2) of the paper and its two ablations
 * (the rows "w/o H2" and "w/o H1" of the score ablation table). */
enum {
    LAZYEV_SCORE_H1_PLUS_H2 = 0,            /* Eq. (2) as printed */
    LAZYEV_SCORE_H1_ONLY = 1,               /* ablation: without the H2-score */
    LAZYEV_SCORE_H2_ONLY = 2,               /* ablation: without the H1-score */
    LAZYEV_SCORE_H1_PLUS_H2_DECREASING = 3  /* Eq. (2) with H2 = 2 sigma(-(MRI - 1)): falls with MRI, as Section 4's
                                               prose and the appendix on the score's formulation require */
};

/*
 * Create a handle.  The seven parameters are the method's: model shape, KV
 * budget B, observation window W and importance threshold alpha (Section 4 of
 * the paper; Algorithm 1's inputs W, B, alpha).  Defaults after create: batch 1,
 * protected recent tokens = window and no protected initial tokens (the paper's
 * rule), automatic eviction on, score = H1 + H2, max_prefill = budget.
 * Errors: EINVAL for head_dim != 128, q_heads not a multiple of kv_heads, more
 * than 8 query heads per KV head, non-positive sizes, budget <= window,
 * threshold < 0 or NaN.
 */
int lazyev_create(lazyev_t** handle, int layers, int q_heads, int kv_heads, int head_dim,
                  int budget, int window, float threshold);

/* Configuration; all of these must come before lazyev_bind() except set_budget,
 * set_auto_evict, set_splits, set_stages and set_groups, which may be called at any time. */
int lazyev_set_batch(lazyev_t* h, int batch);
/* Tokens never evicted: the n_recent newest (paper: W) and the n_initial oldest
 * (paper: 0).  EINVAL unless n_recent >= 1 and budget > n_recent + n_initial. */
int lazyev_set_protect(lazyev_t* h, int n_recent, int n_initial);
/* Longest prompt that will be prefilled; raises the capacity when > budget. */
int lazyev_set_max_prefill(lazyev_t* h, int n_tokens);
/* Budget B_t used by the next evictions; n_recent + n_initial < budget_now <= create-time budget. */
int lazyev_set_budget(lazyev_t* h, int budget_now);
/* on != 0: lazyev_decode_step() runs the eviction itself when one is due (default). */
int lazyev_set_auto_evict(lazyev_t* h, int on);
int lazyev_set_score_mode(lazyev_t* h, int mode);
/* Number of thread blocks (one cluster) that share one unit in the decode
 * kernel: 0 = choose automatically, else 1..8. */
int lazyev_set_splits(lazyev_t* h, int splits);
/* Depth of the decode kernel's shared-memory page ring: 0 = as deep as fits, else 2..6. */
int lazyev_set_stages(lazyev_t* h, int stages);
/* Groups of four consumer warps per block in the decode kernel (each group works on
 * a page of its own): 0 = choose automatically, else 1 or 2. */
int lazyev_set_groups(lazyev_t* h, int groups);

/* on != 0 (default): when a step's decode launch gives every thread block exactly one unit -- problems
 * of up to one unit per SM, where a step is a few microseconds and launch latency decides -- the new
 * token is written into the cache inside that launch (by the warp that streams the token's page)
 * instead of by a launch of its own.  Results are identical either way. */
int lazyev_set_fused_append(lazyev_t* h, int on);

/* Bytes the caller must provide to lazyev_bind(); any output pointer may be NULL. */
int lazyev_query_sizes(const lazyev_t* h, size_t* kv_bytes, size_t* state_bytes, size_t* scratch_bytes);

/*
 * Attach caller-owned device memory (each region at least the size reported by
 * lazyev_query_sizes and 256-byte aligned) and a CUDA stream (cudaStream_t
 * passed as void*, NULL = the legacy default stream).  Zeroes the pool, builds
 * the identity page table and clears the state; asynchronous on the stream.
 * Errors: EINVAL (null / misaligned), ESTATE (already bound), ECUDA.
 */
int lazyev_bind(lazyev_t* h, void* kv_pool, void* state, void* scratch, void* cuda_stream);

/* Replace the page table: host array [units * pages_per_unit] holding a
 * permutation of 0 .. units*pages_per_unit-1.  Only between bind and prefill. */
int lazyev_set_page_table(lazyev_t* h, const int32_t* host_table);

/*
 * Load the prompt's keys and values: device pointers, bf16,
 * [layers, batch, kv_heads, n_tokens, head_dim].  Sets TS = 0, MRI = 0,
 * position = 0..n_tokens-1 and the step counter t = 0.
 * Errors: ESTATE (not bound, or already prefilled), EINVAL, ECAPACITY
 * (n_tokens > max_prefill).
 */
int lazyev_prefill(lazyev_t* h, const void* k, const void* v, int n_tokens);

/*
 * Forget the cached sequences and make the handle ready for a new prompt (lazyev_prefill,
 * lazyev_prefill_observed or lazyev_load_state) on the same memory, configuration and stream:
 * t and n return to 0, budget_now to the create-time budget, the device status word is
 * cleared; the page table is kept.  Asynchronous on the bound stream.  (The paper processes
 * one generation at a time; a server reuses the cache memory for the next batch of requests.)
 * Errors: ESTATE (not bound), ECUDA.
 */
int lazyev_reset(lazyev_t* h);

/*
 * Prompt load WITH observation.  The paper tracks recurrence while decoding and does not say
 * how TS and MRI of prompt tokens start; lazyev_prefill() takes TS = 0, MRI = 0.  This call
 * takes the other reading: tracking (Eq. 1, Algorithm 1's per-token loop) starts at the first
 * prompt token.  Row j of the prompt attends causally over rows 0..j with its own queries
 * (Appendix A, Eq. (attn)), every token's probability is averaged over the query heads of the
 * group, and the statistics are updated in row order at time j - (n_tokens - 1), so the last
 * prompt row is time 0 and decode steps continue at t = 1; a prompt token starts at TS = its
 * own time, MRI = 0.  No eviction happens during the prompt.  The stored probabilities are
 * those of the last prompt row.
 *   q, out : [n_tokens][layers, batch, q_heads, head_dim] bf16 (row-major by prompt position:
 *            row j is laid out like the q / out of lazyev_decode_step); out receives the
 *            causal attention output of every prompt row
 *   k, v   : as for lazyev_prefill()
 * Two implementations (lazyev_set_prompt_mode): LAZYEV_PROMPT_TILED (default) is one launch of
 * a tiled causal-attention kernel on the tensor cores that reads K / V once per tile of query
 * rows; it wants q, k, v and out 16-byte aligned.  LAZYEV_PROMPT_REPLAY pushes the prompt
 * through the decode kernel one row per launch (n_tokens launches over 1..n_tokens cached
 * tokens); it is kept as a cross-check.  Their probabilities agree to float32 rounding, not
 * bit for bit.  Errors as for lazyev_prefill(), plus EINVAL for misaligned pointers.
 */
int lazyev_prefill_observed(lazyev_t* h, const void* q, const void* k, const void* v, int n_tokens, void* out);

enum { LAZYEV_PROMPT_TILED = 0, LAZYEV_PROMPT_REPLAY = 1 };
int lazyev_set_prompt_mode(lazyev_t* h, int mode);
/*
 * Diagnostics for lazyev_prefill_observed(): when device_rows != NULL the next prompt pass also
 * writes, for units [unit_begin, unit_begin + unit_count), the group-mean probability of every
 * token at every prompt row: device_rows[(u * n_tokens + j) * n_tokens + i] for i <= j (float32,
 * caller-owned device memory of unit_count * n_tokens^2 floats; entries with i > j are left
 * untouched).  NULL switches it off.  The tracking of the prompt consumes exactly these values.
 */
int lazyev_set_prompt_dump(lazyev_t* h, float* device_rows, int unit_begin, int unit_count);

/*
 * How long a kernel waits on one of its internal barriers (a page that never arrives, a peer
 * block that never answers) before it gives up, sets the device status word and ends: default
 * 2 s, settable between 0.1 ms and 60 s.  A kernel that gave up leaves the context usable;
 * lazyev_synchronize() then returns EDEVICE and lazyev_reset() clears the word.
 */
int lazyev_set_wait_limit(lazyev_t* h, double seconds);
/*
 * Diagnostics for the time-out path (no counterpart in the paper): with pages >= 0, the warp
 * that feeds a decode block's shared-memory page ring issues no copy beyond its first `pages`
 * pages, so the block's other warps wait for a page that never comes, give up after the wait
 * limit and flag the device status word.  Nothing faults: the kernel ends by itself, and the
 * outputs and statistics of that step are undefined (lazyev_reset() before the handle is used
 * again).  Honoured by launches with one block per unit (lazyev_set_splits(h, 1)); -1 = off.
 * The tiled prompt kernel of lazyev_prefill_observed() honours it too: the thread that feeds a
 * block's ring of key tiles issues no copy beyond its first `pages` key tiles, with the same outcome.
 */
int lazyev_debug_starve_page_ring(lazyev_t* h, int pages);

/*
 * One decode step for all units (Algorithm 1 without its last branch unless
 * automatic eviction is on):
 *   t += 1; the new token (k_new, v_new) is appended with TS = t, MRI = 0;
 *   out = softmax(q K^T / sqrt(head_dim)) V over all cached tokens (Eq. attn);
 *   each cached token's probability, averaged over the query heads of its KV
 *   group, is stored; tokens whose probability is >= threshold get
 *   MRI = max(MRI, t - TS), TS = t (Eq. 1).
 * q, out: [layers, batch, q_heads, head_dim]; k_new, v_new: [layers, batch,
 * kv_heads, head_dim]; all device pointers, bf16.
 * Errors: ESTATE (no prefill), ECAPACITY (cache full: eviction was disabled
 * and never called), EINVAL (automatic eviction is on and this step's eviction
 * would run over more candidates than lazyev_evict() supports), ECUDA.  All of
 * these are found before anything is queued: the step did not happen and may
 * be retried after the cause is removed.  The one exception is ECUDA from a
 * kernel launch: the launches of a step are queued one after the other, so a
 * launch failure leaves the handle in an undefined state (destroy it).
 * Failures that kernels detect (a bounded wait that
 * gave up, an index out of range) are recorded in a device status word and
 * reported by lazyev_synchronize() and lazyev_dump_state() as EDEVICE.
 */
int lazyev_decode_step(lazyev_t* h, const void* q, const void* k_new, const void* v_new, void* out);

/* The same step with HOST buffers (pinned memory recommended; pageable memory works but
 * serialises the copies): copies the inputs to the device, runs the step, copies `out` back and
 * synchronises.  Queries and outputs move in unit ranges on two internal copy streams
 * (created at the first call) while the decode launches of the other ranges run. */
int lazyev_decode_step_host(lazyev_t* h, const void* q, const void* k_new, const void* v_new, void* out);

/*
 * The same step with host buffers, without waiting for it: the call queues the uploads, the
 * step and the download of `out` and returns.  Two steps may be in flight at once; the inputs
 * of step t + 1 are uploaded while the kernels of step t run, and the output of step t comes
 * back while step t + 1 runs, so a caller that has the next inputs ready (another micro-batch,
 * a replayed trace) pays for the copies only where they exceed the kernel time.  A call that
 * finds two steps in flight first waits for the older one.  The host buffers of a step belong
 * to the library until lazyev_host_wait() says the step is complete: q, k_new and v_new must
 * not change and `out` must not be read before that.  Errors as for lazyev_decode_step().
 * (The paper decodes one sequence batch synchronously; this is a serving convenience.)
 */
int lazyev_decode_step_host_async(lazyev_t* h, const void* q, const void* k_new, const void* v_new, void* out);
/* Blocks until at most `in_flight_allowed` (0 or 1) of the steps queued with
 * lazyev_decode_step_host_async() are incomplete: with 1, everything but the newest step is
 * finished and its `out` may be read.  Errors: EINVAL, ECUDA. */
int lazyev_host_wait(lazyev_t* h, int in_flight_allowed);

/*
 * Fork: make `dst` hold an exact copy of the sequences cached in `src` (pool pages, page table,
 * TS, MRI, positions, probabilities, counters, t, n, budget_now), device to device, ordered
 * after everything queued on src's stream and asynchronous on dst's stream (src's stream in
 * turn waits for the copy before it runs anything queued later).  Both handles must
 * be bound on the same device with the same shape, budget, window and protection settings;
 * dst must hold no cache yet (fresh or reset).  Afterwards the two handles decode
 * independently and, given the same inputs, identically.  (No counterpart in the paper; used to
 * branch a generation and to check one entry point against another on the same state.)
 * Errors: EINVAL (different configurations), ESTATE, ECUDA.
 */
int lazyev_copy_state(lazyev_t* dst, lazyev_t* src);

/*
 * Lagged eviction (Section 4 "MRI-Centric Eviction", Eq. 2, Eq. evic): if t is
 * a multiple of the window and n > budget_now, score every unprotected token,
 * keep the budget_now - n_recent - n_initial best (ties: the more recent
 * token) plus the protected ones, and compact K, V, TS, MRI and positions to
 * the front of each unit in generation order; n becomes budget_now.
 * Otherwise does nothing and returns 0.  `*evicted` (optional) receives the
 * number of tokens removed per unit.
 * Limit: the selection keeps one 64-bit key per unprotected token in shared memory, so an
 * eviction over more than 25 600 unprotected tokens per unit returns EINVAL and changes
 * nothing (a cache that never evicts may be longer).  Other errors: ESTATE (no prefill), ECUDA.
 */
int lazyev_evict(lazyev_t* h, int* evicted);

/*
 * lazyev_evict() with its work lists inside the library.  (The paper has no counterpart; this
 * is a deployment convenience.)
 *
 * Who needs it: code that runs where device allocation is off the table -- a plug-in inside a
 * serving process that hands out one fixed arena at start-up and treats any later cudaMalloc
 * as a bug (an allocation synchronises the whole device and stalls every other stream), or a
 * tool attached to a process whose memory pool is already exhausted by the KV cache itself.
 * Such a caller can still provide the pool and the state (they are the method's inputs and
 * outputs), but wants the eviction's work lists to come from somewhere else.
 *
 * This entry point does exactly what lazyev_evict() does -- same trigger test, same kernels,
 * same results bit for bit, same profiling records -- but keeps the source lists and
 * first-moved indices (the part of the scratch region that grows with units * budget) in an
 * array that is compiled into the library (4 MiB + 32 KiB of device memory on every GPU that
 * loads the library, held until the process exits).  It calls no device allocator of any kind.
 * lazyev_bind() still wants a scratch region of the size lazyev_query_sizes() reports (the
 * staging buffers and the 256 KiB table of H2 terms live there); a caller that only ever uses
 * this entry point may leave its first units * budget * 4 bytes untouched by anything else.
 *
 * Limits: units <= 4096 and units * budget_now <= 1,048,576 (2^20) source indices; a larger
 * handle gets LAZYEV_ECAPACITY and a message naming both numbers, before anything runs.
 * The device bound to the handle must be the current device (ESTATE otherwise).
 * The first call on each device looks up the array's device address (one
 * cudaGetSymbolAddress call; the CUDA runtime may load the library's static data at that moment,
 * which is when the 4 MiB show up in the device's memory in use); make that first call outside
 * any stream capture.  Later calls leave the amount of device memory in use unchanged.
 * All handles and all calls on one GPU share the one array and it keeps whatever the last
 * call left in it.  Nothing in it has to start at zero: the select kernel rewrites every entry
 * that the compact kernel reads.  Two evict_static calls whose kernels overlap on the GPU
 * (different streams, no dependency between them) race on the array; order them.
 */
int lazyev_evict_static(lazyev_t* h, int* evicted);

typedef struct lazyev_info {
    int layers, batch, q_heads, kv_heads, head_dim, units;
    int budget, budget_now, window, n_recent, n_initial;
    int capacity;        /* slots per unit (multiple of 64)                  */
    int pages_per_unit;
    int t;               /* decode steps done                                */
    int n;               /* cached tokens per unit                           */
    int prefill;         /* prompt length                                    */
    int splits;          /* blocks per unit used by the last decode launch   */
    int stages;          /* pipeline stages used by the last decode launch   */
    int groups;          /* consumer warp groups used by the last decode launch */
    int tail_units;      /* units of a partly filled last round, given to a second launch (0 = none) */
    int tail_splits;     /* blocks per unit in that second launch                  */
    int grid;            /* blocks launched by the last decode launch        */
    int smem_bytes;      /* dynamic shared memory of the last decode launch  */
    long long launches;  /* kernels launched by this handle so far           */
    long long evictions; /* eviction events so far                           */
    int host_ranges;     /* unit ranges (decode launches) the last lazyev_decode_step_host call was split into */
} lazyev_info_t;

int lazyev_get_info(const lazyev_t* h, lazyev_info_t* out);

/*
 * Event counters kept on the device (tests and diagnostics); synchronises the stream.  They
 * count since lazyev_bind() or the last lazyev_reset().  The selection of an eviction
 * (Appendix A, Eq. (evic)) has two routes per unit: when no more than k candidates have a
 * non-zero score the k-th score is 0 and only the tie rule is left (select_zero_cut_units);
 * otherwise a radix select over the score bits finds the k-th score (select_radix_units).
 */
typedef struct lazyev_counters {
    int device_status;            /* the kernels' status word (0 = healthy)      */
    int select_radix_units;
    int select_zero_cut_units;
} lazyev_counters_t;

int lazyev_get_counters(lazyev_t* h, lazyev_counters_t* out);

/*
 * Snapshot for tests and checkpoints; synchronises the stream.  The caller
 * fills unit_begin / unit_count and the host pointers it wants (NULL = skip);
 * arrays are [unit_count][capacity] (k, v: [unit_count][capacity][head_dim],
 * de-swizzled bf16 bits), valid in the first `n` slots of each unit.
 * `score` receives Eq. (2) evaluated now, at step t, for every cached token.
 * `device_status` is the kernels' status word (0 = healthy).
 */
typedef struct lazyev_dump {
    int unit_begin, unit_count;                 /* in  */
    int t, n, capacity, device_status;          /* out */
    int32_t* pos;
    int32_t* ts;
    int32_t* mri;
    float* pbar;
    double* score;
    uint16_t* k;
    uint16_t* v;
} lazyev_dump_t;

int lazyev_dump_state(lazyev_t* h, lazyev_dump_t* dump);

/*
 * Resume from a snapshot taken with lazyev_dump_state (checkpoint / restore; the paper has
 * no counterpart, its method keeps no state beyond TS and MRI of Eq. (1) and the cache).
 * Valid on a bound handle instead of lazyev_prefill().  `snap` must cover all units
 * (unit_begin = 0, unit_count = units) with pos, ts, mri, k and v set (host arrays laid out
 * as dump_state writes them, row stride snap->capacity; pbar optional, score ignored) and
 * its n and t; `prefill` is the prompt length of the original run (positions of new tokens
 * continue from prefill + t).  The handle may have another capacity than the one the
 * snapshot came from as long as n fits.  Decoding then continues exactly as the original
 * handle would have.  Synchronises the stream; a slow path (one host-to-device copy per page).
 * Errors: EINVAL (partial snapshot, sizes), ESTATE (not bound, or already holds a cache), ECUDA.
 */
int lazyev_load_state(lazyev_t* h, const lazyev_dump_t* snap, int prefill);

/*
 * Distribution of the recurrence intervals in the live cache (Section 4, "Discussion about
 * the choice of W and alpha": the paper sets W to the MRI value below which 80 % of the
 * tokens fall, found offline).  host_hist[b], b < bins - 1, receives the number of cached
 * tokens of units [unit_begin, unit_begin + unit_count) whose MRI equals b (b = 0: never
 * re-activated); host_hist[bins - 1] the number with MRI >= bins - 1.  2 <= bins <= 65536;
 * host_hist is a host array of `bins` 64-bit counts.  Synchronises the stream.
 * Errors: EINVAL (range, bins, null), ESTATE (before prefill), ECUDA.
 */
int lazyev_mri_histogram(lazyev_t* h, int unit_begin, int unit_count, long long* host_hist, int bins);

/*
 * The rule above as one call: *value = the smallest v such that at least `fraction` (in
 * (0, 1]) of the re-activated tokens (MRI >= 1) of the unit range have MRI <= v; 0 when no
 * token has been re-activated yet.  *recurring (may be NULL) = how many such tokens there are.
 * Whether the paper's 80 % counts all tokens or only re-activated ones is not stated; counting
 * only re-activated ones keeps the value meaningful when most tokens never recur.
 */
int lazyev_mri_quantile(lazyev_t* h, int unit_begin, int unit_count, double fraction, int* value, long long* recurring);

/*
 * Per-kernel timing for benchmarks.  While profiling is on, every kernel launch
 * is bracketed by CUDA events on the bound stream (this adds a little latency
 * between kernels, so headline timings are taken with profiling off).  Times are
 * summed per kernel; `*_bytes` are the ALGORITHMIC bytes of the same launches:
 *   decode  : units * (n * (512 + 4) + 2 * group * 256)  -- K/V rows read once,
 *             one float probability written per token, queries read, outputs written
 *   select  : units * (8 * candidates + 4 * budget)       -- TS, MRI read; source list written
 *   compact : moved rows * (2 * (512 + 12) + 4)           -- rows and their state read and written
 * lazyev_get_profile() synchronises the stream; reset != 0 clears the sums.
 */
typedef struct lazyev_profile {
    double append_ms, decode_ms, select_ms, compact_ms;
    double decode_bytes, select_bytes, compact_bytes, compact_rows;
    long long append_launches, decode_launches, select_launches, compact_launches;
} lazyev_profile_t;

int lazyev_set_profiling(lazyev_t* h, int on);
int lazyev_get_profile(lazyev_t* h, lazyev_profile_t* out, int reset);

/* Waits for the stream (and for steps queued with lazyev_decode_step_host_async) and reads the device
 * status word: 0, EDEVICE or ECUDA. */
int lazyev_synchronize(lazyev_t* h);

/* Frees the host-side handle.  Device memory stays with the caller. */
int lazyev_destroy(lazyev_t* h);

/* Bit 0: the library was compiled with -DLAZYEV_DEBUG_BOUNDS: every slot, page-table and work-list
 * index in the kernels is range-checked, a failed check sets bit 1 of the device status word and the
 * access is skipped (slower; for tests -- the release build has none of these checks). */
int lazyev_build_flags(void);

const char* lazyev_strerror(int code);
const char* lazyev_last_error(const lazyev_t* h);

#ifdef __cplusplus
}
#endif
#endif /* LAZYEV_H */
