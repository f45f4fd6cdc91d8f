/*
 * seqsched.h -- C ABI of the sequence-scheduling decode engine for NVIDIA B200 (sm_100a).
 *
 * What the library computes.  The hot path that the paper's sequence scheduling speeds up
 * (arXiv 2305.13144, Sec. 4.1 and Fig. 1 right): a group of queries is sorted by predicted
 * response length, cut into micro-batches, and every micro-batch is decoded greedily by a
 * LLaMA-style decoder (prompt pass, then one token per step with a key/value cache) until
 * all of its rows have finished or the batch's token cap is reached; rows cut by the cap
 * are collected and regenerated at the end of the group.
 *
 * Conventions
 *   - Every function returns an int: SS_OK (0) or a negative SS_ERR_* code.  Nothing throws,
 *     aborts or traps across this boundary.  ss_strerror() gives text.
 *   - "host" / "device" is stated for every pointer.  The caller owns every buffer it passes.
 *     The library owns only the opaque ss_ctx, and it never allocates device memory: all of
 *     its device state (repacked weights, key/value pages, work space) is carved out of the
 *     device arena handed to ss_create().
 *   - All device work is enqueued on the stream given to ss_create() (a cudaStream_t passed
 *     as void*).  Functions are asynchronous with respect to the device unless stated.
 *   - One ss_ctx must be used from one thread at a time.
 *   - Matrices are row-major; projection weights are [out_features, in_features] bf16.
 *   - A response length counts its end-of-sequence token.
 */
#ifndef SEQSCHED_H_
#define SEQSCHED_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ss_ctx ss_ctx;

enum {
  SS_OK = 0,
  SS_ERR_ARG = -1,            /* null pointer, size out of range, inconsistent arguments   */
  SS_ERR_CAPACITY = -2,       /* an output buffer or the arena is too small; nothing written */
  SS_ERR_KV_BUDGET = -3,      /* the batch does not fit the key/value pool; nothing launched */
  SS_ERR_STATE = -4,          /* call out of order (decode before prefill, weights missing)  */
  SS_ERR_CUDA = -5,           /* a CUDA runtime/driver call failed (see ss_last_cuda_error)  */
  SS_ERR_DEVICE_TIMEOUT = -6, /* a bounded wait inside a kernel expired                      */
  SS_ERR_UNSUPPORTED = -7     /* shape outside what the kernels are written for              */
};

/* Decoder shape.  The paper only says "LLaMA-based" (Sec. 1, Sec. 4.2), so every constant
 * of the textbook definition is explicit here.  Constraints: n_heads*head_dim == d_model,
 * head_dim in {64, 128}, d_model % 64 == 0, d_model <= 8192, d_ffn % 8 == 0. */
typedef struct {
  int32_t n_layers, d_model, n_heads, head_dim, d_ffn, vocab, eos_id;
  float rms_eps, rope_theta;
} ss_model_cfg;

/* Capacity of one context. */
typedef struct {
  int32_t max_batch;          /* rows of the largest micro-batch (<= 256)                     */
  int32_t max_ctx;            /* longest prompt + response of one row, in tokens              */
  int32_t max_prefill_tokens; /* tokens of one prompt-pass chunk (work space is sized by it)  */
  int32_t max_new_tokens;     /* longest response (size of the per-row output slots)          */
  int64_t kv_pool_tokens;     /* tokens the key/value pool must hold (rounded up to pages)    */
} ss_runtime_cfg;

/* Scheduler switches and constants (Sec. 4.1 for the rules, Sec. 4.2 "Experimental Setting"
 * for the constants: cell 50, batch 16, threshold 300, token budget 256*50). */
typedef struct {
  int32_t bin_size;           /* cell size; 1 = no binning                                    */
  int32_t base_batch;         /* B0                                                           */
  int32_t use_vbs;            /* variable batch size on/off                                   */
  int32_t use_fcr;            /* failure collection and recomputation on/off                  */
  int32_t vbs_len_threshold;  /* L >= threshold -> B0                                         */
  int32_t vbs_token_budget;   /* below it: nearest power of two to budget / L                 */
  int32_t min_batch, max_batch;
  int32_t max_new_tokens;
  int32_t vanilla;            /* 1: no scheduling, chunks of B0 in the given order, no cap    */
  int64_t kv_budget_bytes;    /* 0 = unlimited                                                */
  int64_t kv_bytes_per_token;
} ss_sched_cfg;

/* One micro-batch: rows order[first_row .. first_row+n_rows). */
typedef struct {
  int32_t first_row, n_rows, cap, is_recompute;
} ss_batch_desc;

/* One named bf16 tensor handed to ss_load_weights().  Names: "embed" [V,d], "lm_head" [V,d],
 * "final_norm" [d], and for each layer i: "l{i}.attn_norm" [d], "l{i}.wq" "l{i}.wk" "l{i}.wv"
 * "l{i}.wo" [d,d], "l{i}.ffn_norm" [d], "l{i}.w_gate" "l{i}.w_up" [F,d], "l{i}.w_down" [d,F].
 * Vectors use rows = 1. */
typedef struct {
  const char* name;
  const void* data;           /* host or device, bf16 bit patterns, row-major, contiguous     */
  int32_t is_device;
  int64_t rows, cols;
} ss_tensor_desc;

/* Per-step options; every pointer may be NULL. */
typedef struct {
  const int32_t* forced_tokens; /* device [B]: teacher forcing -- the row continues with this
                                   token instead of its own choice (finished rows ignore it) */
  float* dump_logits;           /* device fp32 [B, vocab]: the logits the choice was made on  */
  float* dump_hidden;           /* device fp32 [B, d_model]: residual stream before the last norm */
  int32_t* dump_choice;         /* device int32 [B]: the row's own choice (arg-max or draw), before a forced
                                   EOS or a forced token replaces it; written for active rows only */
} ss_step_opts;

/* Per-batch record written by ss_run_group(). */
typedef struct {
  int32_t first_row, n_rows, cap, is_recompute;
  int32_t steps;              /* tokens generated by the longest-running row (prompt pass = 1) */
  int32_t n_failed;           /* rows cut by the cap and sent to recomputation                 */
  float prefill_ms, decode_ms;/* device time (CUDA events)                                     */
} ss_batch_log;

typedef struct {
  int64_t useful_tokens;      /* sum of the final response lengths                             */
  int64_t row_steps;          /* sum over batches of rows * steps                              */
  int64_t steps;              /* sum over batches of steps                                     */
  int32_t n_batches, n_failed;
  float total_ms, prefill_ms, decode_ms;
  double model_bytes;         /* weight + key/value bytes the decode steps had to move         */
  int64_t kernel_launches;    /* kernels of this library launched                              */
} ss_group_stats;

/* Bytes of device arena ss_create() needs for this model and capacity. */
int ss_arena_bytes(const ss_model_cfg* model, const ss_runtime_cfg* rt, size_t* out_bytes);

/* Creates a context.  dev_arena: device memory, 1024-byte aligned, at least ss_arena_bytes().
 * It must outlive the context.  stream: cudaStream_t.  A decode step is one cooperative launch
 * that needs every SM (one CTA per SM waits on grid-wide barriers), so nothing else should occupy
 * the device while steps run; if the CTAs cannot all be resident the launch fails with SS_ERR_CUDA.
 * SS_ERR_UNSUPPORTED for shapes the kernels do not cover, SS_ERR_CAPACITY for a short arena. */
int ss_create(const ss_model_cfg* model, const ss_runtime_cfg* rt, void* dev_arena, size_t arena_bytes,
              void* stream, ss_ctx** out);
int ss_destroy(ss_ctx* ctx);

/* Copies the tensors into the library's own layout inside the arena (q,k,v stacked into one
 * [3d,d] matrix, gate and up into one [2F,d] matrix).  May be called several times; the
 * context is usable once every tensor of the model has been given.  Synchronous. */
int ss_load_weights(ss_ctx* ctx, const ss_tensor_desc* tensors, int32_t n_tensors);

/* The scheduler of Sec. 4.1 (host only, pure, no GPU).  prompt_len, pred_len: host [n].
 * perm: host [n] or NULL -- the processing order of the vanilla arm (identity if NULL);
 * ignored otherwise.  Writes order (host [n]) and up to batch_cap descriptors.
 *   bin(x)  = clamp(x, 1, max_new) rounded up to a multiple of bin_size
 *   order   = stable ascending sort by bin
 *   batch   = grown row by row while its size fits the allowance of its newest (longest) row
 *             (B0, or under VBS: B0 at L >= threshold, else the power of two nearest to
 *             budget/L clamped to [min_batch, max_batch]) and, if a budget is set, while
 *             size * (longest prompt + cap of the newest row) * kv_bytes_per_token fits it
 *   cap     = use_fcr ? min(largest bin in the batch, max_new) : max_new
 * SS_ERR_CAPACITY if batch_cap is too small (n_batches then holds the number needed). */
int ss_schedule(const ss_sched_cfg* cfg, const int32_t* prompt_len, const int32_t* pred_len,
                const int32_t* perm, int32_t n, int32_t* order, ss_batch_desc* batches,
                int32_t batch_cap, int32_t* n_batches);

/* Starts a micro-batch: allocates key/value pages for B rows (worst case prompt + cap tokens
 * each; SS_ERR_KV_BUDGET before any launch if they do not fit), runs the prompt pass
 * (Sec. 4.1 "Overhead of Length Prediction": keys and values of the instruction tokens) and
 * produces each row's first token.
 *   tokens      host int32, the B prompts packed back to back
 *   cu_seqlens  host int32 [B+1], prefix sums of the prompt lengths (cu_seqlens[0] = 0)
 *   eos_at      host int32 [B] or NULL.  NULL: a row ends when its argmax is eos_id.
 *               Otherwise the EOS logit is left out of every argmax and row r's eos_at[r]-th
 *               generated token (1-based) is overwritten with eos_id.
 *   cap         most tokens a row may generate in this batch, the first one included
 *   first_tokens device int32 [B] or NULL
 * A batch in flight must be released before the next ss_prefill(). */
int ss_prefill(ss_ctx* ctx, const int32_t* tokens, const int32_t* cu_seqlens, int32_t B,
               const int32_t* eos_at, int32_t cap, const ss_step_opts* opts, int32_t* first_tokens);

/* Sampled decoding (Sec. 4.2, "Experimental Setting": the paper generates at temperature 0.5; Sec. 3.2: the
 * spread of response lengths between generations).  temperature = 0 (the default) is greedy.  With
 * temperature T > 0 the t-th generated token of a row is a draw from softmax(logits / T), taken as
 *     argmax_v ( logit_v / T - log(-log(u_v)) ),   u_v = ((w >> 9) + 0.5) / 2^23,
 * where w is the first output word of Philox4x32-10 (Salmon et al., SC'11) at counter (v, t, row key, 0) and key
 * (seed & 0xffffffff, seed >> 32); ties go to the lowest id and a suppressed EOS is left out.  The draw depends
 * only on (seed, row key, t, logits): a row regenerated from its prompt repeats its tokens.  Applies to
 * every batch started afterwards.  SS_ERR_ARG for a negative or non-finite temperature. */
int ss_set_sampling(ss_ctx* ctx, float temperature, uint64_t seed);

/* Row keys of the NEXT ss_prefill() only (host int32 [n], n = that batch's row count): the third counter word
 * of the draws above.  Without this call the rows of a batch have keys 0, 1, 2, ...; ss_run_group() uses each
 * row's query index.  Infrastructure of the sampling above, no passage of its own. */
int ss_set_row_keys(ss_ctx* ctx, const int32_t* keys, int32_t n);

/* Prompt reuse (App. C of the paper weighs keeping the instruction's keys and values, computed once for the
 * length-perception pass, against recomputing them for the generation; on its 80 GB GPU it recomputes.  Here the
 * paged cache makes keeping them a matter of not returning pages.)
 * ss_keep_prompts(): while a batch started by ss_prefill() is in flight, take over the pages that hold the first
 *   keep_len[r] tokens of row r (2 <= keep_len[r] <= its prompt length) under the caller's id ids[r] (host int32 [B],
 *   distinct); they stay out of the pool after ss_release_batch().  An id kept before is replaced.
 * ss_resume(): starts a batch of B rows from kept prompts instead of a prompt pass: row r stands one token before
 *   the end of kept prompt ids[r], feeds that token again and produces its first token with an ordinary decode step
 *   (so a resumed batch needs cap decode steps where a prefilled one needs cap - 1).  eos_at, cap, opts,
 *   first_tokens as for ss_prefill().  SS_ERR_STATE if an id is not kept, SS_ERR_KV_BUDGET if the pages for the rest
 *   of the rows' contexts do not fit.  The kept pages stay kept: a row can be resumed again (recomputation).
 * ss_drop_prompts(): returns kept pages to the pool (n = -1: all of them).  Not while a batch is in flight.
 * ss_set_prompt_cache(): what ss_run_group() / ss_run_batches() do with the above: 0 nothing (default); 1 keep the
 *   first keep_len[q] tokens of every query q they process (keep_len host int32 [n], copied); 2 start every batch
 *   whose queries all have a kept prompt with ss_resume(). */
int ss_keep_prompts(ss_ctx* ctx, const int32_t* ids, const int32_t* keep_len);
int ss_resume(ss_ctx* ctx, const int32_t* ids, int32_t B, const int32_t* eos_at, int32_t cap, const ss_step_opts* opts,
              int32_t* first_tokens);
int ss_drop_prompts(ss_ctx* ctx, const int32_t* ids, int32_t n);
int ss_set_prompt_cache(ss_ctx* ctx, int32_t mode, const int32_t* keep_len, int32_t n);

/* One decode step for every active row (App. D: one token per step against the cached keys
 * and values): feed the row's last token at its next position, append its key/value, attend
 * over the row's own cache (per-row length; finished rows are skipped), project, pick the
 * next token (ties -> lowest id).  A row stops being active once it emitted eos_id or
 * generated `cap` tokens; inactive rows report eos_id.
 *   next_tokens     device int32 [B] or NULL
 *   n_active_host   host (pinned) int32 or NULL: number of rows still active after this step,
 *                   valid after the stream has been synchronised */
int ss_decode_step(ss_ctx* ctx, const ss_step_opts* opts, int32_t* next_tokens, int32_t* n_active_host);

/* Enqueues `n_steps` decode steps back to back (no options, no per-step outputs). */
int ss_decode_steps(ss_ctx* ctx, int32_t n_steps, int32_t* n_active_host);

/* Copies the batch's results to the host (synchronises the stream).
 *   out_tokens host int32 [B * stride]: row r's tokens at out_tokens[r*stride ..]
 *   out_len    host int32 [B]: tokens generated
 *   out_status host uint8 [B]: 1 = finished with EOS, 0 = cut by the cap */
int ss_read_batch(ss_ctx* ctx, int32_t* out_tokens, int32_t stride, int32_t* out_len, uint8_t* out_status);

/* Returns the batch's pages to the pool. */
int ss_release_batch(ss_ctx* ctx);

/* The whole group (Fig. 1 right; Sec. 4.1): schedule, run every micro-batch (prompt pass,
 * decode until all rows finished or the cap), collect the rows the cap cut, regenerate them
 * from their prompts in batches of B0 with cap = max_new.  Synchronous; all arguments host.
 *   prompt_tokens / prompt_off [n+1]   packed prompts
 *   pred_len [n], perm [n] or NULL     as for ss_schedule
 *   eos_at [n] or NULL                 as for ss_prefill
 *   out_tokens / out_off [n+1]         caller-sized slots (slot i holds at least max_new)
 *   out_len [n], out_status [n]        final length; 1 = EOS, 0 = truncated at max_new
 *   order [2n]                         processing order; entries n.. list the failures
 *   log [log_cap], n_log               one record per batch, first pass then recomputation
 *   stats                              may be NULL */
int ss_run_group(ss_ctx* ctx, const ss_sched_cfg* cfg, const int32_t* prompt_tokens, const int64_t* prompt_off,
                 const int32_t* pred_len, const int32_t* perm, const int32_t* eos_at, int32_t n,
                 int32_t* out_tokens, const int64_t* out_off, int32_t* out_len, uint8_t* out_status,
                 int32_t* order, ss_batch_log* log, int32_t log_cap, int32_t* n_log, ss_group_stats* stats);

/* Runs a given list of micro-batches on this context, one after the other (the body of ss_run_group() without its
 * scheduling): the unit of work when the batches of one schedule are dealt to several GPUs (Sec. 1: batches of
 * different perceived lengths can go to different GPU nodes; each GPU holds a replica of the weights and no data
 * crosses between GPUs while batches run).  Synchronous; all arguments host.
 *   prompt_tokens / prompt_off [n+1], eos_at [n] or NULL   the whole group, as for ss_run_group
 *   order [n_order], batches [n_batches]                    batch i = queries order[first_row .. first_row + n_rows)
 *   out_tokens / out_off [n+1], out_len [n], out_status [n] written for the rows that ended here (not for failures)
 *   fail_rows [n], n_fail                                   queries the cap cut (cap < max_new, no EOS), in batch
 *                                                           and row order: the caller requeues them
 *   log [log_cap], n_log, stats                             as for ss_run_group (stats may be NULL) */
int ss_run_batches(ss_ctx* ctx, const ss_sched_cfg* cfg, const int32_t* prompt_tokens, const int64_t* prompt_off,
                   const int32_t* eos_at, int32_t n, const int32_t* order, int32_t n_order, const ss_batch_desc* batches,
                   int32_t n_batches, int32_t* out_tokens, const int64_t* out_off, int32_t* out_len, uint8_t* out_status,
                   int32_t* fail_rows, int32_t* n_fail, ss_batch_log* log, int32_t log_cap, int32_t* n_log,
                   ss_group_stats* stats);

/* Deals micro-batches to n_gpus replicas (host only, pure).  The paper only proposes the hand-out (Sec. 1); the
 * rule here: estimated cost of a batch = cap * (weight_bytes + rows * (mean prompt length + cap / 2) *
 * kv_bytes_per_token) in integer arithmetic; batches in order of decreasing cost (ties: lower index) each go to the
 * replica with the smallest total so far (ties: lowest replica).  gpu_of: host int32 [n_batches] (output). */
int ss_deal_batches(const ss_batch_desc* batches, int32_t n_batches, const int32_t* order, const int32_t* prompt_len,
                    int64_t weight_bytes, int64_t kv_bytes_per_token, int32_t n_gpus, int32_t* gpu_of);

/* Bytes a decode step must move (weights once, plus the cached keys/values of the active
 * rows, plus the entries written); host arithmetic on lengths the caller supplies:
 * ctx_len host [B] (tokens cached before the step), active host uint8 [B]. */
int ss_step_model_bytes(const ss_ctx* ctx, const int32_t* ctx_len, const uint8_t* active, int32_t B, double* out);

/* (The paper has no counterpart to this call; it exists for integration.)
 * The LM-head projection for callers that cannot allocate device memory: code running while
 * its framework captures a CUDA graph, inside an allocator callback, in a process whose device
 * memory is all handed to another pool, or in a loop where an allocation's hidden
 * synchronisation is not acceptable.  Computes, with the same kernels as the engine,
 *     logits[r][v] = sum_i lm_head[v][i] * bf16( hidden[r][i] * rsqrt(mean_j hidden[r][j]^2 + eps) * gain[i] )
 *   hidden    device fp32 [n_rows, d_model]      norm_gain device bf16 [d_model]
 *   lm_head   device bf16 [vocab, d_model], 16-byte aligned
 *   logits    device fp32 [n_rows, vocab] (output)      stream  cudaStream_t
 * No ss_ctx, no arena: the two temporaries (bf16 activations, fp32 split-K partial sums) live in
 * an 8 MiB array that is part of the library image, so every GPU that loads the library holds
 * those 8 MiB until the process ends.  The call itself allocates nothing on the device or the
 * host.  Limits: n_rows <= 16, d_model <= 8192 and a multiple of 64, and vocab small enough for
 * the partial sums to fit (vocab 32000 uses 3.7 MiB; on a 148-SM part a vocab of about 94000 is
 * the edge); beyond them SS_ERR_CAPACITY is returned and nothing is launched.
 * The first call on each device looks up the array's device address and raises the kernel's
 * shared-memory limit; make that first call, with the device current, before any stream capture.
 * All calls share the one array and it keeps what the last call left there (the call clears the
 * only word that must start at zero), so two calls whose kernels may overlap on the GPU --
 * different streams, or threads -- race; keep calls on one device in one stream order.
 * The call is asynchronous: it returns once its three kernels are enqueued.  SS_ERR_CUDA means a
 * launch was refused (an error that the caller's earlier work left pending is discarded on entry
 * and not reported here).  Should a bounded wait inside the projection kernel give up, every
 * element of `logits` is set to NaN instead of a sum of incomplete partials. */
int ss_logits_noalloc(const float* hidden, const void* norm_gain, const void* lm_head, int32_t n_rows,
                      int32_t d_model, int32_t vocab, float rms_eps, float* logits, void* stream);

/* Failure detection.  Every wait inside a kernel (on a barrier between the SMs, on a copy, on the tensor
 * cores) is bounded: when the limit runs out the kernel records which wait it was, all of its roles leave, and the
 * next ss_read_batch() / ss_run_group() returns SS_ERR_DEVICE_TIMEOUT (once; the context is then usable again).
 * ss_set_wait_limit_ms() sets that limit (default about 2000 ms; 1..60000).
 * ss_selftest_wait_timeout() demonstrates the path without putting any work at risk: it launches one small
 * kernel in which every SM waits, for at most limit_us microseconds, for an arrival that never comes, and returns
 * what the runtime then reports -- SS_ERR_DEVICE_TIMEOUT when detection works.  SS_ERR_STATE while a batch is in
 * flight.  Infrastructure, no passage of the paper. */
int ss_set_wait_limit_ms(ss_ctx* ctx, int32_t ms);
int ss_selftest_wait_timeout(ss_ctx* ctx, int32_t limit_us);

/* Tracing (App. D measures per-token time; this shows where one decode step spends it).  Off by default;
 * ss_set_trace(ctx, 1) makes every following decode step record its stage boundaries. */
int ss_set_trace(ss_ctx* ctx, int32_t on);

/* Copies the time stamps (nanoseconds of the GPU's global timer) that CTA 0 took during the LAST decode step:
 * out[0] start, out[1] first operand ready, then for each projection in execution order
 * (qkv, o, gate/up, down per layer, LM head) four stamps: own accumulators drained, all partials
 * visible, own share of the following stage done, stage complete on every SM.
 * out: host uint64 [cap]; n receives the number of stamps (2 + 4 * (4 * n_layers + 1));
 * SS_ERR_CAPACITY if cap is smaller, SS_ERR_STATE if tracing is off.  Synchronises the stream. */
int ss_step_trace(ss_ctx* ctx, uint64_t* out, int32_t cap, int32_t* n);

const char* ss_strerror(int code);
/* Last device status word (0 = clean; non-zero = which bounded wait expired). Synchronises. */
int ss_last_device_status(ss_ctx* ctx, uint32_t* out);
/* Last CUDA error code seen by this context (cudaError_t or CUresult as int). */
int ss_last_cuda_error(const ss_ctx* ctx);
/* Kernels launched by this context so far. */
int64_t ss_kernel_launches(const ss_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* SEQSCHED_H_ */
