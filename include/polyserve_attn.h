/*
 * polyserve_attn.h -- C ABI of the mixed-batch paged-KV attention library.
 *
 * One serving-instance iteration batches every running decode request with a
 * dynamically sized chunk of prefill tokens (paper section 2.4, chunked
 * prefill; section 4.7, dynamic chunking).  The attention step of that
 * iteration is Softmax(Q K^T / sqrt(d)) V over the K, V of all previous tokens
 * (section 2.1), per request, with the K, V held in a paged cache addressed
 * through a block table.  The scheduler predicts iteration time from a profiled
 * table keyed by token batch size and KV-cache size (section 4.5); the sweep
 * entry point below emits that table for the attention step.
 *
 * Notation: request r has prior[r] >= 0 tokens attended in earlier iterations
 * and q_len[r] >= 1 new tokens; kv_len[r] = prior[r] + q_len[r].  New token i
 * of request r attends keys 0 .. prior[r] + i (itself included).  Q head h
 * reads KV head h / (n_q_heads / n_kv_heads).  All kv_len[r] tokens' K and V,
 * the new ones included, are in the cache before ps_attn_run is called.
 *
 * Conventions
 *   - every function returns a ps_status; nothing throws across the boundary;
 *   - "host" / "dev" in a parameter name says where the pointer must live;
 *   - streams are cudaStream_t passed as void* (NULL = the default stream);
 *   - the caller owns Q, out, block table, workspace and (optionally) the pool
 *     memory; the library owns the handles it returns;
 *   - no entry point synchronises the device unless its comment says so;
 *   - the library targets sm_100a only and has no CPU path: without a usable
 *     device every launching call returns PS_ERR_CUDA.
 */
#ifndef POLYSERVE_ATTN_H_
#define POLYSERVE_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PS_OK = 0,
    PS_ERR_INVALID = 1,     /* bad argument (null pointer, negative length, q_len < 1, ...) */
    PS_ERR_OOM = 2,         /* host or device allocation failed */
    PS_ERR_CUDA = 3,        /* a CUDA runtime call failed; see ps_last_error() */
    PS_ERR_UNSUPPORTED = 4, /* shape outside what the kernels handle */
    PS_ERR_WORKSPACE = 5,   /* workspace smaller than the plan requires */
    PS_ERR_BOUNDS = 6,      /* device saw a page id outside the pool */
    PS_ERR_TIMEOUT = 7      /* a bounded device-side wait expired */
} ps_status;

/* Attention geometry.  Supported: head_dim in {64, 128}, page_size == 16,
 * n_q_heads a multiple of n_kv_heads (1, 2, 4 or 8 q heads per kv head).
 * dtype == 0: bf16 K/V cache (bf16 in, fp32 accumulate, bf16 out).
 * dtype == 1: the cache holds K and V as FP8 E4M3 codes with one fp32 scale per
 * (token, kv head) and tensor -- scale = amax / 448 over the head_dim values,
 * rounded up to 8 significant bits (1 for an all-zero vector), code = x /
 * scale rounded to nearest even and
 * saturated at +-448, both divisions IEEE fp32; a stored token never changes
 * when later tokens are appended.  Q and out stay bf16, accumulation fp32; the
 * decode kernel multiplies with f16 operands (E4M3 converts to f16 exactly), so
 * Q is clamped to +-65504 and V scales are meant to lie in [2.4e-7, 255].  The
 * paper states no precision (its section 3.3 only notes that decode attention
 * time is set by the bytes of KV cache read); this variant halves those bytes.
 * It exists for head_dim 128 and serves decode rows only: ps_attn_plan refuses
 * batches with q_len > 1 and ps_profile_grid sweeps the bf16 cache only. */
typedef struct {
    int32_t n_q_heads;
    int32_t n_kv_heads;
    int32_t head_dim;
    int32_t page_size;
    int32_t dtype;
} ps_shape;

typedef struct ps_kv ps_kv;     /* paged K/V pool                       */
typedef struct ps_plan ps_plan; /* work partition of one batch of lengths */

/* Planner options; a NULL pointer or a zero field selects the default. */
typedef struct {
    int32_t decode_segment_tokens;  /* KV tokens per decode work item (multiple of page_size); 0 = auto */
    int32_t prefill_segment_tokens; /* KV tokens per prefill work item (multiple of 128); 0 = auto */
    int32_t num_sms;                /* SM count to balance for; 0 = ask the current device */
} ps_plan_opts;

/* ------------------------------------------------------------------------ */
/* Paged KV pool (the paged cache and block table of section 6.1's serving    */
/* engines; cache population of section 2.1).                                 */
/* ------------------------------------------------------------------------ */

/* Bytes a pool of num_pages pages occupies. */
ps_status ps_kv_bytes(const ps_shape *shape, int64_t num_pages, size_t *bytes_out);

/*
 * Create a pool of num_pages pages of page_size tokens.  If dev_mem is NULL
 * the library allocates the pool with cudaMalloc and frees it in ps_kv_free;
 * otherwise dev_mem (device memory, 1024-byte aligned, dev_bytes >=
 * ps_kv_bytes()) stays owned by the caller and must outlive the handle.  The
 * physical layout inside a page is private to the library: fill the pool with
 * ps_kv_write and read it back with ps_kv_gather.  Pool contents are not
 * initialised.  Which pages a sequence uses is the caller's decision, passed
 * in as the block table.
 */
ps_status ps_kv_alloc(const ps_shape *shape, int64_t num_pages, void *dev_mem, size_t dev_bytes, ps_kv **out);
ps_status ps_kv_free(ps_kv *kv);

/*
 * Scatter the K, V of new tokens into their pages (section 2.1: each pass
 * populates the KV cache).  k_new_dev / v_new_dev: bf16 [T, n_kv_heads,
 * head_dim], T = sum q_len, requests in batch order, tokens in order.  Token i
 * of request r goes to logical position prior_host[r] + i, i.e. page
 * block_table_dev[r * max_pages + pos / page_size], slot pos % page_size.
 * Asynchronous on `stream`; lengths are read before the call returns.
 * Errors: PS_ERR_INVALID for null pointers, q_len < 1, prior < 0 or a position
 * beyond max_pages * page_size; page ids outside the pool are skipped on the
 * device and reported by ps_kv_status.
 */
ps_status ps_kv_write(ps_kv *kv, const void *k_new_dev, const void *v_new_dev, const int32_t *block_table_dev,
                      int32_t max_pages, const int32_t *prior_host, const int32_t *q_len_host, int32_t n,
                      void *stream);

/*
 * Copy logical tokens [0, len) of one sequence out of the pool, bit for bit,
 * into contiguous bf16 [len, n_kv_heads, head_dim] buffers (either may be
 * NULL).  block_table_row_dev: that sequence's page ids (device).  Asynchronous.
 */
ps_status ps_kv_gather(const ps_kv *kv, const int32_t *block_table_row_dev, int32_t len, void *k_out_dev,
                       void *v_out_dev, void *stream);

/*
 * FP8 pools (dtype == 1): ps_kv_write takes the same bf16 inputs and quantises
 * them as ps_shape describes; ps_kv_gather returns the codes, one byte per
 * element ([len, n_kv_heads, head_dim] uint8 in k_out_dev / v_out_dev).
 * ps_kv_gather_fp8 returns codes and the fp32 scales ([len, n_kv_heads]); any
 * output may be NULL.  Together they let a test compare the stored cache bit
 * for bit with a reference quantiser.  PS_ERR_INVALID on a bf16 pool.
 */
ps_status ps_kv_gather_fp8(const ps_kv *kv, const int32_t *block_table_row_dev, int32_t len, void *k_codes_out_dev,
                           void *v_codes_out_dev, float *k_scale_out_dev, float *v_scale_out_dev, void *stream);

/* Synchronises `stream`, then returns PS_OK or PS_ERR_BOUNDS for the pool's
 * write/gather kernels since the last call, and clears the flag. */
ps_status ps_kv_status(ps_kv *kv, void *stream);

/* ------------------------------------------------------------------------ */
/* Work partition (host only).                                                */
/* ------------------------------------------------------------------------ */

/*
 * Partition one batch into work items.  Rows with q_len == 1 are decode rows
 * (memory-bound KV streaming, section 2.2); rows with q_len > 1 are prefill
 * chunks (dense contraction, section 3.4).  A chunk of at most 8 tokens whose
 * context is short enough to re-read (q_len * kv_len * bytes per token <= 32
 * MB) is run as q_len decode rows instead -- token i as a row that sees
 * prior + i + 1 keys of the same sequence -- in batches whose decode rows
 * hold at most 128 MB of K/V and whose plan does not force prefill segments:
 * there the prefill kernel's launch costs more than the re-reads.  Its items
 * then appear among the decode items.  Long contexts are cut into KV
 * segments whose partial results are combined afterwards (decode rows inside
 * the decode kernel, prefill items by a merge kernel).  Host arrays
 * prior_host / q_len_host have n entries and are read before the call returns.
 * max_pages_per_seq is the row stride of the block table later given to
 * ps_attn_run; kv_len[r] must not exceed max_pages_per_seq * page_size.
 *
 * *plan_inout == NULL creates a plan; otherwise the existing plan is rebuilt
 * in place, reusing its pinned staging memory (the call first waits until the
 * plan's last ps_attn_run has finished reading that memory).  Running the
 * device is not needed: the only CUDA calls are pinned-memory management and,
 * if opts->num_sms == 0, a device-attribute query.
 * *workspace_bytes_out: device bytes ps_attn_run needs for this plan.
 * Errors: PS_ERR_INVALID (n < 1, q_len < 1, prior < 0, kv_len too long),
 * PS_ERR_UNSUPPORTED (shape), PS_ERR_OOM.
 */
ps_status ps_attn_plan(const ps_shape *shape, const int32_t *prior_host, const int32_t *q_len_host, int32_t n,
                       int32_t max_pages_per_seq, const ps_plan_opts *opts, ps_plan **plan_inout,
                       size_t *workspace_bytes_out);
ps_status ps_plan_free(ps_plan *plan);

/* Counts describing a plan, for tests and reports. */
typedef struct {
    int32_t n_decode_items;
    int32_t n_prefill_items;
    int32_t n_merge_rows;      /* (token, q head) outputs combined from several KV segments */
    int32_t decode_segment_tokens;
    int32_t prefill_segment_tokens;
    int64_t n_partial_slots;   /* fp32 partial rows held in the workspace */
    int64_t total_q_tokens;
    int32_t n_launches;        /* kernels one ps_attn_run launches for this plan */
    int32_t decode_sms;        /* SMs the decode kernel is sized for */
    int32_t prefill_sms;       /* SMs the prefill kernel is sized for; in a mixed batch the two kernels run side by
                                  side on disjoint SMs when that is predicted to be faster (decode_sms + prefill_sms
                                  = all SMs), otherwise one after the other on all of them */
} ps_plan_info;
ps_status ps_plan_get_info(const ps_plan *plan, ps_plan_info *info_out);

/*
 * Copy the plan's work items to host arrays for inspection (tests check that
 * the items cover every (row, q head, visible key) exactly once).  Each item is
 * 8 int32: {request, kv_head, key_begin, key_end, q_token, n_tokens,
 * partial_slot, first_position}.  q_token is the packed index of the item's
 * first q token, n_tokens how many consecutive q tokens it covers (1 for
 * decode, at most 256 / G for prefill), partial_slot is -1 when the item writes final output, and
 * first_position = prior + index of its first token in the chunk.  Either
 * output may be NULL; capacities are in items.
 */
ps_status ps_plan_get_items(const ps_plan *plan, int32_t *decode_items_out, int64_t decode_capacity,
                            int32_t *prefill_items_out, int64_t prefill_capacity);

/* ------------------------------------------------------------------------ */
/* Attention for one iteration.                                               */
/* ------------------------------------------------------------------------ */

/*
 * out[t, h, :] = sum_j softmax_j(q[t, h, :] . K[j, g, :] / sqrt(d)) V[j, g, :]
 * over the keys the token may see (section 2.1).  q_dev / out_dev: bf16
 * [T, n_q_heads, head_dim] packed as for ps_kv_write; lse_out_dev: optional
 * fp32 [T, n_q_heads], natural-log sum of exponentials of the scaled scores
 * (NULL to skip).  block_table_dev: int32 [n, max_pages_per_seq] page ids;
 * entries past a sequence's last page are never read.  workspace_dev: device
 * memory (256-byte aligned) of at least the plan's workspace bytes; its
 * contents need no initialisation and are scratch.  Asynchronous on `stream`:
 * the work list is uploaded (on a stream of the plan's own, ordered against
 * `stream` with events, into one of two slots of the workspace so that it can
 * run under the previous run's kernels), then the prefill, decode and merge
 * kernels run; for a batch with both row classes the decode kernel may run on
 * a second stream of the plan, beside the prefill kernel on disjoint SMs (the
 * merge kernel then follows the prefill kernel at once, under the decode
 * kernel), and is joined back into `stream` before the call's work is
 * complete in stream order.
 * Ordering rule for the workspace: all runs that use one workspace -- of one
 * plan, re-planned or not, and of different plans that take turns on it --
 * must be issued to the same stream, or be ordered by the caller.  Under that
 * rule no host synchronisation is needed between a ps_attn_plan / ps_attn_run
 * pair and the next, whatever the batches: the two work-list slots sit at
 * fixed strides that only grow, a run's upload waits for the run two calls
 * ago that used its slot, and whenever the library cannot rely on that record
 * (first use of the memory, slots moved because a work list outgrew them,
 * another plan's run on the workspace in between) the upload is instead
 * ordered behind everything already on `stream`.
 * The call may be made while `stream` is being captured into a CUDA graph:
 * the upload then becomes a node of the graph on `stream` (each replay copies
 * the plan's staging image again) and the graph replays this plan, with these
 * pointers, as often as wanted.  The graph belongs to the plan as it was
 * captured: after ps_attn_plan on the same plan object capture again, and do
 * not re-plan or free the plan while a replay is in flight.
 * Returns host-detectable errors only (PS_ERR_INVALID, PS_ERR_WORKSPACE,
 * PS_ERR_CUDA); errors seen on the device are read with ps_plan_status.
 */
ps_status ps_attn_run(ps_plan *plan, const ps_kv *kv, const void *q_dev, const int32_t *block_table_dev,
                      void *out_dev, float *lse_out_dev, void *workspace_dev, size_t workspace_bytes,
                      void *stream);

/* Synchronises `stream`, then reports what the plan's last run saw on the
 * device: PS_OK, PS_ERR_BOUNDS (a page id outside the pool, which was skipped,
 * or a work record pointing outside the batch, which was not followed; the
 * output is invalid) or PS_ERR_TIMEOUT (a bounded wait expired; output is
 * invalid).  The status word lives in the workspace: read it before another
 * plan runs on the same workspace. */
ps_status ps_plan_status(ps_plan *plan, void *stream);

/*
 * Bound, in nanoseconds, of every wait inside this plan's kernels (for a bulk
 * copy to land, for another warp's hand-over, for a group of MMAs to retire).
 * A wait that runs out sets the run's status to PS_ERR_TIMEOUT; the warps of
 * that CTA stop, let the copies and MMAs already in flight finish (bounded
 * again, by a fixed second), release their tensor memory and return, so the
 * context stays usable and nothing is left waiting.  Default: 2 s; at most
 * 4 s (PS_ERR_INVALID beyond, or for a negative value).  Zero makes
 * a wait give up as soon as it finds its phase incomplete -- in practice the
 * first wait of every CTA -- which is how the tests reach this path on a
 * healthy device.  Takes effect at the next ps_attn_run (a captured graph
 * keeps the value it was captured with).
 */
ps_status ps_plan_set_wait_limit(ps_plan *plan, int64_t limit_ns);

/*
 * ps_attn_run without a caller-provided workspace.  (The paper has no
 * counterpart for this call; it exists for integration reasons only.)
 *
 * Some callers cannot hand the library device memory at the moment they need
 * attention: a plug-in running inside a host engine that owns every byte of
 * HBM and forbids cudaMalloc after start-up, a latency-critical loop where an
 * allocation would stall the device, or a process whose memory budget is fixed
 * when it loads.  For them the scratch that ps_attn_run takes as
 * `workspace_dev` (the uploaded work list and the split-KV partial results
 * passed from the decode / prefill kernels to the merge kernel) lives in a
 * fixed array of PS_STATIC_WORKSPACE_BYTES inside the library's device image.
 * Every GPU that loads the library keeps that array until the process exits.
 *
 * Arguments and results are those of ps_attn_run; inputs, outputs, pool and
 * plan are still the caller's.  This call itself allocates nothing, on the
 * host or on the device (the plan was allocated earlier by ps_attn_plan).
 * A plan whose workspace need exceeds PS_STATIC_WORKSPACE_BYTES is refused
 * with PS_ERR_WORKSPACE before anything is launched: use ps_attn_run, or
 * smaller batches.
 *
 * The first call on each device looks up the array's device address (a
 * runtime query made with that device current, as it must be at every call);
 * make that first call before starting any stream capture.  All calls on a
 * device share the one array and it keeps whatever the last call left there:
 * each run rewrites the header words that must start at zero.  The array is a
 * workspace like any other and ps_attn_run's ordering rule applies to it:
 * issue all calls on a device to one stream (plans may then take turns freely;
 * the library orders each upload behind the other plan's run), or order them
 * yourself -- runs that overlap on the GPU would overwrite each other's work
 * list and partials.  Read ps_plan_status before another plan uses the array.
 */
#define PS_STATIC_WORKSPACE_BYTES (8u << 20)
ps_status ps_attn_run_static(ps_plan *plan, const ps_kv *kv, const void *q_dev, const int32_t *block_table_dev,
                             void *out_dev, float *lse_out_dev, void *stream);

/*
 * Per-kernel timing of the next runs of this plan (the profile of section 4.5
 * split into its prefill-attention and decode-attention terms, section 3.4).
 * ps_plan_set_timing(plan, max_runs) makes each of the next max_runs calls of
 * ps_attn_run record CUDA events around the prefill, decode and merge launches
 * (on the stream each is launched on; max_runs = 0 switches recording off;
 * when the two kernels of a mixed batch run side by side their intervals
 * overlap and each is longer than the kernel would take alone); calling it again
 * restarts the count.  ps_plan_get_timing synchronises `stream` and returns
 * the mean duration in milliseconds of each kernel over the runs recorded so
 * far, and how many there were.  A kernel the plan does not launch reports the
 * (near-zero) gap between its two events.
 */
ps_status ps_plan_set_timing(ps_plan *plan, int32_t max_runs);
ps_status ps_plan_get_timing(ps_plan *plan, void *stream, float *prefill_ms_out, float *decode_ms_out,
                             float *merge_ms_out, int32_t *n_runs_out);

/* ------------------------------------------------------------------------ */
/* Latency-table sweep (section 4.5: a profiled map from batch size and KV    */
/* cache size to execution time, which the scheduler consults).               */
/* ------------------------------------------------------------------------ */

typedef struct {
    const int32_t *chunk_sizes;   int32_t n_chunk_sizes;   /* prefill chunk tokens; 0 = no chunk */
    const int32_t *decode_counts; int32_t n_decode_counts; /* decode rows per batch */
    const int32_t *mean_ctxs;     int32_t n_mean_ctxs;     /* mean context length m */
    int32_t seeds_per_cell;       /* independent length draws per cell */
    int32_t warmup;               /* untimed runs per draw (>= 1) */
    int32_t iters;                /* timed runs per draw (>= 1) */
    uint64_t seed_base;           /* draw s of cell c uses seed seed_base + seeds_per_cell * c + s */
    int32_t include_kv_write;     /* != 0: each timed run first appends the batch's new tokens with ps_kv_write
                                     (section 2.1: the pass that computes attention also populates the cache) */
    double hbm_peak_gbs;          /* denominators of the rows' roofline_frac: memory bandwidth in GB/s and dense bf16 */
    double bf16_peak_tflops;      /* tensor rate in TFLOP/s, e.g. as measured on the device; 0 = nominal 8000 / 2250 */
} ps_grid_spec;

typedef struct {
    int32_t chunk, n_decode, mean_ctx, seed_index;
    uint64_t seed;
    int32_t token_batch;      /* chunk + n_decode: the table's "batch size" key */
    int32_t prefill_prior;    /* prior context drawn for the chunk */
    int64_t kv_tokens;        /* sum of kv_len: the table's "KV cache size" key */
    double decode_bytes;      /* kv_len * bytes of K+V per token, summed over decode rows */
    double prefill_flops;     /* 4 d Hq (c prior + c (c + 1) / 2) */
    float latency_us;         /* median over iters of one ps_attn_run, CUDA events */
    float latency_min_us;
    float latency_max_us;
    float plan_us;            /* host time of ps_attn_plan for this draw */
    float decode_TBps;        /* decode_bytes / latency: the decode-attention term of section 3.4 as a rate */
    float prefill_TFLOPs;     /* prefill_flops / latency (both rates are over the whole step, so in a mixed batch
                                 each is a lower bound on what its kernel reached) */
    float roofline_frac;      /* max(decode_bytes / hbm peak, prefill_flops / bf16 peak) / latency: 1 means the step
                                 took what its slower resource needs when the two kernels overlap perfectly */
} ps_grid_row;

/*
 * Time ps_attn_run over chunk_sizes x decode_counts x mean_ctxs x seeds.
 * Per draw: decode contexts (kv_len) are integers uniform on [m/2, 3m/2], the
 * chunk's prior context is one more draw of that law; pages are assigned by a
 * seeded permutation of a pool with 25 % spare pages.  Lengths come from
 * SplitMix64 streams keyed by the draw's seed, so a caller can regenerate
 * them.  K, V and Q hold bounded pseudo-random bf16 values; small batches
 * rotate over several copies of the pool so that no run finds its KV in L2.
 * The library allocates and frees all device memory it needs (largest cell x
 * rotation) and synchronises the device; `stream` is used for the timed runs.
 * rows (host, capacity max_rows) receives one row per draw in sweep order
 * (chunk-major, then decode count, then mean context, then seed);
 * *n_rows_out is the count written.  If csv_path is not NULL the rows are also
 * written there as CSV with a header line (first column: "attn", or
 * "attn+kv_write" when the append is inside the timed region).
 * Errors: PS_ERR_INVALID (null/empty spec, max_rows too small),
 * PS_ERR_UNSUPPORTED, PS_ERR_OOM, PS_ERR_CUDA; a device-side error of any run
 * aborts the sweep with that status.
 */
ps_status ps_profile_grid(const ps_shape *shape, const ps_grid_spec *spec, ps_grid_row *rows, int64_t max_rows,
                          int64_t *n_rows_out, const char *csv_path, void *stream);

/* Thread-local text of the last error returned on this thread ("" if none). */
const char *ps_last_error(void);
const char *ps_version(void);

#ifdef __cplusplus
}
#endif
#endif /* POLYSERVE_ATTN_H_ */
