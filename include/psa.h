/*
 * psa -- parallel-sample shared-prefix decode attention for NVIDIA B200 (sm_100a).
 *
 * One decode step of attention for B samples that were all drawn from the same few
 * prompts: the paper's learning loop samples N candidate answers per task from ONE
 * prompt made of selected demonstrations plus the task (Algorithm 1, the sampling
 * step; appendix "Experiment details": 64 samples per temperature, at most 1024
 * output tokens).  Every sample s of prompt p owns one query vector per query head and
 * attends, unmasked, to the L_p prompt tokens it shares with its siblings followed by
 * its own S_s generated tokens:
 *
 *     out[s,h,:] = softmax_j( sm_scale * q[s,h,:] . k_j ) . v_j ,   lse = ln sum_j exp(...)
 *
 * which is the operator of the paper's "attn" benchmark group, softmax(S).V with
 * S = QK^T (appendix "Benchmark details").  The library evaluates it in three device
 * stages and one host stage:
 *
 *   plan    (host)   cut prefix and suffix work into pieces that fill every SM
 *   prefix  (device) all samples x heads of a KV head batched against the shared prefix
 *                    K/V, read once; deferred-division online softmax (the paper's
 *                    attn Task 2 recurrence) on tensor cores
 *   suffix  (device) per-sample attention over ragged, paged K/V
 *   merge   (device) log-sum-exp combination of every row's partial results
 *
 * Conventions
 *   - "host" / "device" after a pointer says where the memory lives.  Every buffer is
 *     caller-owned.  The library owns only the opaque plan (host memory).
 *   - bf16 means the upper 16 bits of an IEEE-754 binary32, stored as uint16_t.
 *   - Query head h reads KV head h / G, G = num_q_heads / num_kv_heads.
 *   - Samples of prompt 0 come first in q/out/lse, then prompt 1, ...; prompts are packed
 *     back to back along the token axis of prefix_k / prefix_v.
 *   - No function throws, aborts or traps.  Host-detectable problems come back as a
 *     status code; device-side problems (a bounded wait that ran out) are written to a
 *     status word in the workspace, the affected outputs are left unwritten, and
 *     psa_check_status reports them.
 *   - Supported: head_dim in {64, 128}; G in {1, 2, 4, 8}; page_size 16; sm_scale > 0.
 *     Anything else is PSA_ERR_UNSUPPORTED.  There is no fallback path of any kind.
 */
#ifndef PSA_H_
#define PSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct psa_plan psa_plan_t;

typedef enum {
    PSA_OK = 0,
    PSA_ERR_INVALID_ARG = 1, /* null pointer, negative length, misaligned buffer, ... */
    PSA_ERR_UNSUPPORTED = 2, /* shape or dtype outside the supported set */
    PSA_ERR_WORKSPACE = 3,   /* workspace missing, too small, or not bound to this plan */
    PSA_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed */
    PSA_ERR_TIMEOUT = 5,     /* device: a bounded wait expired; outputs of that block unwritten */
    PSA_ERR_BOUNDS = 6       /* device: an index outside its table was met and skipped */
} psa_status_t;

enum { PSA_OUT_BF16 = 0, PSA_OUT_F32 = 1 };

typedef struct {
    int32_t num_q_heads;
    int32_t num_kv_heads;
    int32_t head_dim;   /* 64 or 128 */
    int32_t page_size;  /* tokens per page of the suffix pool: 16 */
    float   sm_scale;   /* multiplies q.k before the softmax; > 0 */
    int32_t out_dtype;  /* PSA_OUT_BF16 or PSA_OUT_F32 */
    int32_t num_sms;    /* SMs to plan for; 0 = ask the current CUDA device */
    int32_t suffix_chunk_tokens;   /* tokens per suffix work item: 0 = planner's choice, else a multiple of 64 */
    int32_t prefix_tiles_per_item; /* 128-key tiles per prefix work item: 0 = planner's choice */
    int32_t prefix_rows_per_item;  /* query rows per prefix work item: 0 = planner's choice, else 128 or 256 */
    int32_t prefix_kernel;         /* which prefix block shape to launch: PSA_PREFIX_KERNEL_AUTO (0) = planner's choice */
} psa_config_t;

/* Prefix block shapes (psa_config_t.prefix_kernel); a tuning knob like the three above, results are the same.
 * Items of more than 128 query rows always take a two-row-tile shape (DECOUPLED unless COUPLED is asked for); the
 * others apply to items of at most 128 rows. */
enum {
    PSA_PREFIX_KERNEL_AUTO = 0,
    PSA_PREFIX_KERNEL_SMALL = 1,     /* one row tile, 64-key tiles, small enough to share its SM with a suffix block */
    PSA_PREFIX_KERNEL_LONG = 2,      /* one row tile, 128-key tiles, deep ring: long HBM-bound items of few rows */
    PSA_PREFIX_KERNEL_DECOUPLED = 3, /* two softmax warpgroups fed two score tiles ahead (on alternate key tiles when
                                        there is one row tile); the block owns its SM */
    PSA_PREFIX_KERNEL_COUPLED = 4    /* two row tiles, one score buffer each (the earlier shape, kept for comparison) */
};

/* What the planner decided; for tests, logs and roofline accounting. */
typedef struct {
    int32_t num_sms;
    int32_t num_samples;          /* B */
    int32_t num_prefix_items;     /* prefix work items (one thread block each) */
    int32_t num_suffix_items;     /* suffix work items at the planned suffix lengths */
    int32_t prefix_tile_keys;     /* keys per tensor-core tile (128) */
    int32_t prefix_tiles_per_item;/* upper bound of key tiles in one prefix item */
    int32_t suffix_chunk_tokens;  /* tokens per suffix work item */
    int32_t kernel_launches;      /* device launches one psa_decode enqueues */
    int64_t num_partial_rows;     /* rows of the partial-result arrays in the workspace */
} psa_plan_info_t;

/*
 * Plan stage (part 4 of the design; the paper's "one prompt, many samples" shape is its
 * only input).  Host only; touches CUDA only when cfg->num_sms == 0.
 *   prefix_lens [num_prefixes] host: L_p >= 0.
 *   n_samples_per_prefix [num_prefixes] host: N_p >= 0; B = sum N_p.
 *   suffix_lens [B] host: upper bounds of S_s used to size the work lists.  psa_decode
 *     reads the actual lengths from device memory; each must be <= its bound here.
 * On success *out_plan is a new plan the caller destroys with psa_plan_destroy.
 */
psa_status_t psa_plan_create(const psa_config_t *cfg, int32_t num_prefixes,
                             const int32_t *prefix_lens, const int32_t *n_samples_per_prefix,
                             const int32_t *suffix_lens, psa_plan_t **out_plan);
/*
 * Plan for a CASCADE of shared prefixes: the prompts of the paper's sampling step are themselves layered --
 * base prompt + demonstrations d_j shared by every task, then the task text shared by that task's N samples
 * (Algorithm 1, the sampling step; the prompt composer appends the task-specific input last) -- so the big
 * level can be batched over ALL samples.  A "group" is a run of consecutive tokens of the packed prefix arrays
 * attended by a run of consecutive samples:
 *   group g = tokens [T_g, T_g + group_token_len[g]) with T_g = sum of the earlier groups' lengths,
 *             samples [group_first_sample[g], group_first_sample[g] + group_n_samples[g]).
 * A sample attends to every group that contains it (at most 4) plus its own suffix; the order of keys does
 * not matter to the result.  psa_plan_create is the special case "group p = prompt p, groups do not overlap".
 * All arrays are host memory; num_samples = B.  Everything else (psa_decode, workspaces) is unchanged.
 */
psa_status_t psa_plan_create_cascade(const psa_config_t *cfg, int32_t num_groups, const int32_t *group_first_sample,
                                     const int32_t *group_n_samples, const int32_t *group_token_len, int32_t num_samples,
                                     const int32_t *suffix_lens, psa_plan_t **out_plan);
/*
 * The step before the path: prefill, i.e. causal attention of a prompt over itself (token i attends to tokens
 * 0..i of its prompt), which a decoder runs once per prompt before the samples share the resulting K/V -- and
 * again when demonstrations are added between iterations (section "Stratification and selection").  The same
 * tensor-core kernel serves it: every query token is a row, the 256 / G tokens of a row group share the keys up
 * to the group's last token, and the kernel masks the keys beyond each row's own token.
 *   prompt_lens [num_prompts] host.  Prompts are packed back to back in q / k / v / out / lse.
 * psa_prefill: q [T, Hq, D] bf16, k / v bf16 with element (token t, kv head, d) at t*kv_strides[0] +
 * head*kv_strides[1] + d, out [T, Hq, D] (bf16 or f32 per cfg.out_dtype), lse [T, Hq] f32; T = sum of prompt_lens;
 * all device memory; workspace bound with psa_plan_bind_workspace.  Only enqueues work.
 */
psa_status_t psa_plan_create_prefill(const psa_config_t *cfg, int32_t num_prompts, const int32_t *prompt_lens,
                                     psa_plan_t **out_plan);
psa_status_t psa_prefill(const psa_plan_t *plan, const void *q, const void *k, const void *v, const int64_t kv_strides[2],
                         void *out, float *lse, void *workspace, size_t workspace_bytes, void *cuda_stream);
psa_status_t psa_plan_destroy(psa_plan_t *plan);
psa_status_t psa_plan_get_info(const psa_plan_t *plan, psa_plan_info_t *info);

/* Bytes of device workspace psa_decode needs with this plan (work lists + partial results). */
size_t psa_plan_workspace_bytes(const psa_plan_t *plan);

/*
 * Copy the plan's work lists into `workspace` (device, 256-byte aligned, at least
 * psa_plan_workspace_bytes) and clear its status word.  Enqueued on `cuda_stream`
 * (a cudaStream_t; NULL = default stream).  Call once per (plan, workspace) pair, before
 * the first psa_decode that uses them and before any stream capture.
 */
psa_status_t psa_plan_bind_workspace(const psa_plan_t *plan, void *workspace, size_t workspace_bytes,
                                     void *cuda_stream);

/*
 * Host copies of the work lists, for tests.  Each prefix item is 8 int32:
 *   {first_token (index into the packed prefix), n_keys, kv_head, first_sample,
 *    n_rows (valid query rows = samples x G), partial_row0, prompt, split}
 * each suffix item 4 int32: {sample, kv_head, first_token, partial_row0}.
 * Pass NULL to query the count only.  Returns the number of items.
 */
int32_t psa_plan_prefix_items(const psa_plan_t *plan, int32_t *items8);
int32_t psa_plan_suffix_items(const psa_plan_t *plan, int32_t *items4);

/*
 * One decode step (prefix, suffix and merge stages).  Only enqueues work on
 * `cuda_stream`; never synchronises, never allocates device memory.
 *
 *   q              [B, Hq, D] bf16 device, contiguous, 16-byte aligned.
 *   prefix_k/v     bf16 device, 16-byte aligned; element (token t, kv head, d) at
 *                  t*prefix_strides[0] + head*prefix_strides[1] + d  (elements; D contiguous;
 *                  strides multiples of 8 elements).  May be NULL when every L_p == 0.
 *   suffix_k/v_pool bf16 device, 16-byte aligned; element (page, kv head, slot, d) at
 *                  page*pool_strides[0] + head*pool_strides[1] + slot*pool_strides[2] + d.
 *   page_indptr    [B+1] int32 device: sample s owns page_indices[page_indptr[s] .. page_indptr[s+1]).
 *   page_indices   int32 device: physical page ids; token t of sample s is in its page t/16, slot t%16.
 *   suffix_lens    [B] int32 device: actual S_s, each <= the planned bound (larger is clamped).
 *   out            [B, Hq, D] device, bf16 or f32 per cfg.out_dtype.
 *   lse            [B, Hq] f32 device, natural logarithm; -inf for an empty context (out = 0).
 *   workspace      the buffer bound with psa_plan_bind_workspace.
 * The prefix and suffix stages run side by side; the merge stage, which stream order puts behind the suffix
 * stage only, learns that the prefix stage is complete from two counters kept in the workspace's status area
 * (bounded wait; PSA_ERR_TIMEOUT in the status word if it ever ran out).  The counters belong to the workspace:
 * calls that share one must be ordered on one stream, concurrent calls must use distinct workspaces.
 */
psa_status_t psa_decode(const psa_plan_t *plan, const void *q,
                        const void *prefix_k, const void *prefix_v, const int64_t prefix_strides[2],
                        const void *suffix_k_pool, const void *suffix_v_pool, const int64_t pool_strides[3],
                        const int32_t *page_indptr, const int32_t *page_indices, const int32_t *suffix_lens,
                        void *out, float *lse, void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * psa_decode without a caller workspace and without any allocation.  (The paper has no
 * counterpart for this entry point; it exists for how the library gets embedded.)
 *
 * Who needs it: callers that are not allowed to allocate device memory around a decode step --
 * a plugin inside a serving process whose memory pool already owns the whole GPU, code
 * running under an allocator it does not control, or a latency-critical loop in which a
 * cudaMalloc would stall the device.  The scratch memory of the step (work lists, status
 * word, partial results of the prefix and suffix stages) lives in one fixed array of
 * PSA_STATIC_WORKSPACE_BYTES inside the library image; every GPU that loads the library
 * holds that much memory until the process ends.  This function calls no cudaMalloc,
 * cudaFree or other allocating routine; it copies the plan's work lists into the array
 * (which also clears the status word) and then runs the same three stages as psa_decode,
 * on `cuda_stream`, without synchronising.  All other arguments are those of psa_decode.
 *
 *   - A plan whose psa_plan_workspace_bytes exceeds PSA_STATIC_WORKSPACE_BYTES is rejected
 *     with PSA_ERR_WORKSPACE (the message names both sizes); nothing is launched.
 *   - The first call on each device looks up the array's device address (with that device
 *     current).  Make that first call outside any stream capture.
 *   - When the array's memory is taken: the array belongs to a CUDA module of the library, and
 *     the driver creates it when it loads that module on a device.  Under the runtime's default
 *     lazy module loading that happens inside the FIRST call on the device -- the one call that
 *     can still fail for lack of memory, or take milliseconds; with CUDA_MODULE_LOADING=EAGER it
 *     happens when the library is loaded.  So make one warm-up call per device during
 *     initialisation, before your own pool claims the remaining memory.  From the second call
 *     on, free device memory does not change.
 *   - All calls on a device share the one array, and it keeps what the last call left in
 *     it.  Two calls whose GPU work can overlap (different streams, different threads or
 *     different plans) race on it: serialise them, or give one of them psa_decode with its
 *     own workspace.
 *   - Device-side status: every call clears the status word before its kernels run, so read
 *     it with psa_static_check_status BEFORE the next call if you need it (psa_check_status
 *     cannot: the array's address is private to the library).
 */
#define PSA_STATIC_WORKSPACE_BYTES (16u << 20)
psa_status_t psa_decode_static(const psa_plan_t *plan, const void *q,
                               const void *prefix_k, const void *prefix_v, const int64_t prefix_strides[2],
                               const void *suffix_k_pool, const void *suffix_v_pool, const int64_t pool_strides[3],
                               const int32_t *page_indptr, const int32_t *page_indices, const int32_t *suffix_lens,
                               void *out, float *lse, void *cuda_stream);

/*
 * Companions of psa_decode_static (no counterpart in the paper either).  psa_static_check_status synchronises
 * `cuda_stream`, returns the device-side status word the last psa_decode_static step on the current device left
 * in the library's array (PSA_OK, PSA_ERR_TIMEOUT or PSA_ERR_BOUNDS) and clears it; it allocates nothing.
 * psa_static_selftest_bounded_wait is psa_selftest_bounded_wait reporting into that array, so that the error
 * path can be exercised without a caller workspace.
 */
psa_status_t psa_static_check_status(void *cuda_stream);
psa_status_t psa_static_selftest_bounded_wait(uint64_t limit_ns, void *cuda_stream);

/*
 * The stages one by one, for tests and per-kernel timing.  Same arguments as psa_decode.
 * prefix and suffix write partial results into the workspace; merge reads them.
 */
psa_status_t psa_decode_prefix(const psa_plan_t *plan, const void *q, const void *prefix_k, const void *prefix_v,
                               const int64_t prefix_strides[2], void *workspace, size_t workspace_bytes,
                               void *cuda_stream);
psa_status_t psa_decode_suffix(const psa_plan_t *plan, const void *q, const void *suffix_k_pool,
                               const void *suffix_v_pool, const int64_t pool_strides[3],
                               const int32_t *page_indptr, const int32_t *page_indices, const int32_t *suffix_lens,
                               void *workspace, size_t workspace_bytes, void *cuda_stream);
psa_status_t psa_decode_merge(const psa_plan_t *plan, const int32_t *suffix_lens, void *out, float *lse,
                              void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * The same step with every tensor in HOST memory (pinned memory makes the copies
 * asynchronous): copies the inputs into `staging` (device, psa_decode_host_staging_bytes),
 * runs psa_decode, copies out and lse back to the host buffers, all on `cuda_stream`.
 * num_prefix_tokens / num_pool_pages size the copies; the K/V layouts are the dense
 * defaults ([tokens, Hkv, D] and [pages, Hkv, 16, D]).  Does not synchronise.
 */
size_t psa_decode_host_staging_bytes(const psa_plan_t *plan, int64_t num_prefix_tokens, int64_t num_pool_pages,
                                     int64_t num_page_indices);
psa_status_t psa_decode_host(const psa_plan_t *plan, const void *q_host,
                             const void *prefix_k_host, const void *prefix_v_host, int64_t num_prefix_tokens,
                             const void *suffix_k_pool_host, const void *suffix_v_pool_host, int64_t num_pool_pages,
                             const int32_t *page_indptr_host, const int32_t *page_indices_host,
                             int64_t num_page_indices, const int32_t *suffix_lens_host,
                             void *out_host, float *lse_host, void *staging, size_t staging_bytes,
                             void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Synchronise `cuda_stream` and return the device-side status word of `workspace`
 * (PSA_OK, PSA_ERR_TIMEOUT or PSA_ERR_BOUNDS), then clear it.
 */
psa_status_t psa_check_status(const psa_plan_t *plan, void *workspace, void *cuda_stream);

/*
 * Debug aid (no counterpart in the paper): check a page table against the plan before the suffix stage trusts it.
 * For every sample: 0 <= suffix_lens[s] <= the planned bound, at least ceil(S_s / 16) pages in its list, every
 * page id in [0, num_pool_pages).  Enqueues one small kernel; a violation raises PSA_ERR_BOUNDS in the status
 * word of `workspace` (read it with psa_check_status).  psa_decode itself does not check page ids.
 */
psa_status_t psa_validate_page_table(const psa_plan_t *plan, const int32_t *page_indptr, const int32_t *page_indices,
                                     const int32_t *suffix_lens, int64_t num_pool_pages, void *workspace,
                                     size_t workspace_bytes, void *cuda_stream);

/*
 * The step after the path: append one new token per sample to the paged suffix K/V (each of the paper's samples
 * grows by one token per decode step, up to 1024: appendix "Experiment details").  For every sample s, the rows
 * new_k[s], new_v[s] ([B, Hkv, D] bf16 device, contiguous) are written to position S_s = suffix_lens[s] of the
 * sample's page list and suffix_lens[s] becomes S_s + 1 (device memory, in place), all on `cuda_stream`.
 * The page for position S_s must already be in the sample's page list (a negative id there counts as missing), and
 * S_s must be below the bound the plan was made with; otherwise that sample is left untouched and the status word reports PSA_ERR_BOUNDS
 * (psa_check_status).  The plan itself does not change: psa_decode may follow immediately.
 */
psa_status_t psa_append_kv(const psa_plan_t *plan, const void *new_k, const void *new_v,
                           void *suffix_k_pool, void *suffix_v_pool, const int64_t pool_strides[3],
                           const int32_t *page_indptr, const int32_t *page_indices, int32_t *suffix_lens,
                           void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * psa_append_kv with page allocation on the device.  A sample whose length S_s is a multiple of 16 needs a fresh page for
 * its next token; here the library takes it from a caller-owned stack of free page ids instead of expecting the caller to
 * have put it into the page list beforehand, so that a decode loop (attend, draw, append, ...) can run without the host
 * looking at the lengths -- for instance as one replayed CUDA graph.
 *   page_indptr   [B+1] int32 device: sample s owns the SLOTS page_indices[page_indptr[s] .. page_indptr[s+1]) (its capacity).
 *   page_indices  int32 device, in/out: slots 0 .. ceil(S_s / 16) - 1 of a sample hold its pages; every slot beyond must
 *                 hold a negative value until this function assigns a page to it.
 *   free_pages    int32 device: free_pages[0 .. *free_count) are ids of pages nobody owns (a stack, top at the end).
 *   free_count    int32 device, in/out.
 * Samples are served in sample order, so the result does not depend on scheduling: the r-th sample (in that order) that
 * needs a page gets free_pages[*free_count - 1 - r]; *free_count drops by the number of pages handed out.  When the stack
 * runs out, the remaining samples that need a page are left untouched (length, pools and list unchanged) and the status
 * word reports PSA_ERR_BOUNDS; the same holds for a sample at its planned bound or without a free slot in its list.
 * Everything else is psa_append_kv.  Enqueues two kernels on `cuda_stream`.
 */
psa_status_t psa_append_kv_alloc(const psa_plan_t *plan, const void *new_k, const void *new_v,
                                 void *suffix_k_pool, void *suffix_v_pool, const int64_t pool_strides[3],
                                 const int32_t *page_indptr, int32_t *page_indices, int32_t *suffix_lens,
                                 const int32_t *free_pages, int32_t *free_count,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * The step after the path, second half: draw the next token of every sample from its logits.  The paper samples its
 * candidate answers at temperature T in {0.4, 0.7, 1.0} with a seed (appendix "Experiment details").  Row r gets
 *     tokens[r] = argmax_i ( logits[r, i] / T_r + g_i ),   g_i = -ln(-ln u_i)          (ties: lowest i)
 * (the Gumbel-max identity: token i comes out with probability softmax(logits[r] / T_r)_i); T_r = 0 means greedy
 * decoding, argmax_i logits[r, i].  The uniforms are Philox4x32-10 words (Salmon et al., SC'11): counter
 * (i / 4, step, r, 0), key (low, high word of seeds[r]), u_i = ((word[i % 4] >> 9) + 0.5) * 2^-23, so a draw depends
 * only on (seeds[r], step, r, i): pass the decode step as `step` and keep the seeds fixed to get reproducible runs.
 *
 *   logits        [num_rows, vocab] device, bf16 (PSA_OUT_BF16) or f32 (PSA_OUT_F32) per `logits_dtype`, 16-byte
 *                 aligned, element (r, i) at r*row_stride + i; row_stride >= vocab, a multiple of 8 elements.
 *   temperature   [num_rows] f32 device (<= 0 or NaN: greedy);  seeds [num_rows] u64 device.
 *   tokens        [num_rows] int32 device, out.
 *   scratch       device, 8-byte aligned, psa_sample_scratch_bytes(num_rows) bytes; caller-owned, cleared and
 *                 overwritten by every call (calls that share it must be ordered on one stream).
 * Arithmetic is fp32 (scores are compared in fp32).  Only enqueues work (a memset and two kernels) on `cuda_stream`.
 * num_rows <= 65535.  -inf logits are never drawn unless the whole row is -inf (then token 0); NaN logits are
 * not supported.
 */
size_t psa_sample_scratch_bytes(int32_t num_rows);
psa_status_t psa_sample_tokens(const void *logits, int32_t logits_dtype, int64_t row_stride, int32_t num_rows, int32_t vocab,
                               const float *temperature, const uint64_t *seeds, uint32_t step, int32_t *tokens,
                               void *scratch, size_t scratch_bytes, void *cuda_stream);
/*
 * psa_sample_tokens with the decode step kept in DEVICE memory: the kernels read *step_device where psa_sample_tokens
 * takes `step`, and add `advance` to it once every row has been drawn.  A CUDA graph that holds this call can so be
 * replayed step after step and still draw fresh, reproducible numbers (the paper's samples run for up to 1024 steps:
 * appendix "Experiment details").  step_device: 4-byte aligned device pointer, in/out.  Everything else as above.
 */
psa_status_t psa_sample_tokens_at(const void *logits, int32_t logits_dtype, int64_t row_stride, int32_t num_rows, int32_t vocab,
                                  const float *temperature, const uint64_t *seeds, uint32_t *step_device, uint32_t advance,
                                  int32_t *tokens, void *scratch, size_t scratch_bytes, void *cuda_stream);

/*
 * The paper's three "attn" tasks (appendix "Benchmark details"): softmax(S) V folded over a stream of keys in the
 * three forms the paper asks its agents to implement -- task 0 "MaxSum" (running maximum and sum, output normalised at
 * every step), task 1 "ExpMaxDiff" feeding "DivSum" (maximum split from the sum, still normalised every step), task 2
 * "ExpMaxDiff" feeding two weighted sums divided once at the end (the form the fast kernels above use).  Plain
 * CUDA-core reference kernels (one warp per row, one key at a time, fp32), for small problems: they tie the library to
 * the paper's operator forms, they are not a fast path.
 *   q [num_rows, head_dim], k, v [num_keys, head_dim]: bf16 device, contiguous; scores are sm_scale * q.k_j.
 *   out [num_rows, head_dim] f32, m_out, l_out [num_rows] f32: the output and the final running maximum and sum
 *   (natural exponent; lse = m + ln l).  No keys: out = 0, m = -inf, l = 0, the paper's initial state.
 * head_dim a multiple of 32, at most 256.  Only enqueues one kernel on `cuda_stream`.
 */
psa_status_t psa_attn_task(int32_t task, const void *q, const void *k, const void *v, int32_t num_rows, int32_t num_keys,
                           int32_t head_dim, float sm_scale, float *out, float *m_out, float *l_out, void *cuda_stream);

/*
 * Self-test of the device-side error path (no counterpart in the paper).  Enqueues one tiny kernel whose only
 * wait is on a barrier that nothing completes; the wait gives up after `limit_ns` (<= 1 s), the kernel writes
 * PSA_ERR_TIMEOUT into the status word of `workspace` and exits normally.  psa_check_status then reports and
 * clears it, and the context stays usable.  This is how the bounded waits of the prefix stage fail, too.
 */
psa_status_t psa_selftest_bounded_wait(void *workspace, size_t workspace_bytes, uint64_t limit_ns, void *cuda_stream);

const char *psa_status_string(psa_status_t status);
const char *psa_last_error_message(void); /* thread-local detail of the last non-OK return */
int32_t psa_version(void);

#ifdef __cplusplus
}
#endif
#endif /* PSA_H_ */
