/*
 * as_verify.h - C ABI of the batched verification step of speculative decoding on one B200.
 *
 * The step this library implements is the one the paper states in Sec. 2.2 (draft several tokens,
 * verify them with the target model in one pass, lossless) and Sec. 3
 * (D(b) drafted tokens per step, a per-request rejection rate), fed by the per-request draft lengths
 * L_i that Sec. 4.2 / Eq. 3 / Algorithm 2 allocate: request i of a batch brings k_i >= 0 draft
 * tokens (a single chain) and the target model scores k_i + 1 positions in one batched pass.
 * The paper leaves the numerics of that pass open; the readings this library takes are written
 * beside each call.
 *
 * Notation.  B requests.  Request i has n_i committed KV entries (positions 0..n_i-1) and k_i
 * drafts.  Its rows are j = 0..k_i: row 0 is the last emitted token (position n_i), row j >= 1 is
 * draft j (position n_i + j).  cu_q[i] = sum_{i'<i}(k_i'+1), cu_d[i] = sum_{i'<i} k_i',
 * total_q = cu_q[B], total_d = cu_d[B].  Hq query heads, Hkv KV heads, G = Hq/Hkv, head dim D,
 * page size bs tokens, vocabulary V.
 *
 * Conventions.  Every function returns an int status (AS_OK = 0).  Nothing throws, aborts or traps.
 * Pointers marked "dev" are device pointers owned by the caller and must stay valid until the work
 * enqueued on `stream` has finished; pointers marked "host" are read before the call returns.
 * The library allocates no device memory: all scratch lives in the workspace the caller binds to
 * the plan (one exception, as_accept_greedy_static, keeps its scratch in a fixed array of the library's
 * device image and needs no plan).  All GPU work is enqueued on the caller's stream (a cudaStream_t passed as void*, NULL =
 * the default stream) and is asynchronous with respect to the host.  A plan must not be used from
 * two host threads at once; distinct plans are independent.  Faults found on the device (a page id
 * outside the pool, a draft token outside the vocabulary, a bounded wait that ran out) set bits in
 * a status word in the workspace, the offending work is skipped, and as_plan_check() reports them.
 */
#ifndef AS_VERIFY_H_
#define AS_VERIFY_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define AS_API __attribute__((visibility("default")))
#else
#define AS_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

enum {
  AS_OK = 0,
  AS_ERR_INVALID_ARG = 1,  /* a null pointer, a negative or out-of-range size, lengths that overflow the plan */
  AS_ERR_UNSUPPORTED = 2,  /* shape outside what the kernels are built for (see as_plan_create)             */
  AS_ERR_WORKSPACE = 3,    /* workspace not bound, misaligned or too small                                   */
  AS_ERR_CUDA = 4,         /* a CUDA runtime / driver call failed; as_last_error() has its message          */
  AS_ERR_DEVICE_FLAG = 5,  /* as_plan_check(): a kernel recorded a fault (see AS_FLAG_*)                     */
  AS_ERR_TIMEOUT = 6       /* as_plan_check(): a bounded device-side wait ran out                            */
};

/* bits of the device status word returned through as_plan_check() */
enum {
  AS_FLAG_BAD_PAGE = 1,    /* block-table entry outside [0, num_blocks) reached by a kernel */
  AS_FLAG_BAD_TOKEN = 2,   /* draft token outside [0, vocab): treated as a rejection        */
  AS_FLAG_WAIT_CAP = 4,    /* a bounded mbarrier wait ran out (2 s); the step is void        */
  AS_FLAG_BAD_ACCEPT = 8,  /* as_kv_commit saw accept_len outside [0, k_i]: clamped         */
  AS_FLAG_BAD_PLAN = 16    /* as_plan_device(): lengths out of range or over capacity: the step is empty */
};

enum { AS_COMMIT_SCRUB = 1 /* zero the rejected slots that stay in held pages */ };

/* attention kernel selection, for as_plan_set_attn_impl() */
enum {
  AS_ATTN_AUTO = 0,   /* tensor-core kernel where the shape allows, else the SIMT kernel */
  AS_ATTN_SIMT = 1,   /* portable fp32 SIMT kernel (any supported shape)                 */
  AS_ATTN_TC = 2      /* tcgen05 / TMA kernel; AS_ERR_UNSUPPORTED if the shape is not covered */
};

/* One attention-layer flavour.  window = 0: full causal attention.  window = W > 0: row at
 * position p sees the W keys p-W+1..p (its own included).  sm_scale = 0 selects 1/sqrt(head_dim).
 * sinks: dev fp32 [num_q_heads] or NULL; a sink logit joins the softmax denominator of every row
 * of its head and carries no value.  (Paper: silent on all of these.) */
typedef struct {
  int32_t num_q_heads, num_kv_heads, head_dim, block_size;
  int32_t window;
  float sm_scale;
  const float* sinks;
} as_layer_desc;

typedef struct as_plan_s as_plan_t;

AS_API const char* as_status_string(int status);
/* Text of the last failure on the calling thread ("" if none).  The pointer stays valid until the
 * next failing call on the same thread. */
AS_API const char* as_last_error(void);

/* Creates a plan for batches of at most max_batch requests with at most max_draft drafts each,
 * block tables of max_blocks_per_req columns, and KV pools of num_blocks pages, on CUDA device
 * `device`.  `kinds` lists the distinct attention flavours of the model (all must share the head
 * counts, head_dim and block_size); as_verify_attn() picks one by index.  The descriptors are
 * copied.  Supported: head_dim in {64, 128}; block_size in {16, 32, 64, 128};
 * num_q_heads a multiple of num_kv_heads with G * (max_draft + 1) <= 256; num_kinds in 1..4.
 * Host-only: allocates host memory, no device memory, launches nothing. */
AS_API int as_plan_create(as_plan_t** out, const as_layer_desc* kinds, int num_kinds, int max_batch, int max_draft,
                   int max_blocks_per_req, int num_blocks, int device);
AS_API int as_plan_destroy(as_plan_t* plan);

/* Bytes of device workspace the plan needs (metadata, split-KV partials, status word). */
AS_API size_t as_plan_workspace_bytes(const as_plan_t* plan);
/* Binds caller-owned device memory (256-byte aligned, at least as_plan_workspace_bytes()).  The
 * plan keeps the pointer until it is destroyed or re-bound; contents need no initialisation. */
AS_API int as_plan_bind(as_plan_t* plan, void* dev_workspace, size_t bytes);
/* Forces one attention kernel (AS_ATTN_*); takes effect at the next as_plan(). */
AS_API int as_plan_set_attn_impl(as_plan_t* plan, int impl);

/* Fixed launches (off by default).  When on, as_plan() lays the step's metadata out at the same workspace
 * addresses in every step and as_verify_attn / as_accept / as_kv_commit size every grid for the plan's
 * maxima (max_batch, max_draft), the kernels taking the step's actual sizes from the workspace.  The
 * arguments and launch shapes of those three calls then depend only on the plan and on the pointers passed
 * to them, so a caller may record them once (stream capture into a CUDA graph) and replay the recording
 * after every later as_plan() of the same plan: as_plan() itself stays outside the recording (it is host
 * work plus one copy on the stream).  Costs one copy of the full metadata capacity per step and some
 * blocks that exit at once; meant for small batches, where a step is bound by launch overhead.  The paper
 * has no counterpart (Sec. 4.2 / Eq. 3 choose the draft lengths anew in every step, which is what this keeps cheap).
 * Takes effect at the next as_plan(). */
AS_API int as_plan_set_fixed_launch(as_plan_t* plan, int on);

/* Ragged-batch metadata for one verify step (the consumer of the draft lengths L_i of Eq. 3).
 *   seq_lens, draft_lens: host int32 [batch]: n_i and k_i (0 <= k_i <= max_draft).
 *   block_table: dev int32 [batch, max_blocks_per_req], -1 = no page.  Must cover positions
 *     0..n_i+k_i of every request when free_blocks is NULL.
 *   free_blocks: host int32 [num_free] or NULL.  When given, the plan assumes request i holds exactly
 *     ceil(n_i/bs) pages and hands out the pages for positions up to n_i+k_i from the front of this
 *     list, in (request, logical page) order, writing them into block_table on the stream;
 *     *num_taken (host, may be NULL) receives how many were used.  Too few -> AS_ERR_INVALID_ARG.
 * Computes cu_q / cu_d, the per-row map, and per layer kind the split-KV work list: the visible
 * keys of all (request, kv-head) pairs are laid end to end and cut into equal shares, one per
 * resident CTA, so that every SM streams the same number of KV bytes; a pair that is cut is merged
 * afterwards in a fixed order (results do not depend on timing).  When a step mixes short and long
 * drafts (head_dim 128, launches not fixed), the requests are bucketed by row count into two such work
 * lists, each run by its own attention launch with the kernel instance of its widest request.  Copies
 * the metadata to the workspace on `stream`.  Integer-only and deterministic. */
AS_API int as_plan(as_plan_t* plan, int batch, const int32_t* seq_lens, const int32_t* draft_lens,
            int32_t* block_table, const int32_t* free_blocks, int num_free, int* num_taken, void* stream);

/* The same step metadata built ON THE DEVICE (one small kernel on `stream`) from length arrays that live in device
 * memory: seq_lens / draft_lens are DEVICE int32 [batch] - e.g. the seq_lens a previous as_kv_commit has just
 * written and draft lengths chosen on the device - and free_blocks is a DEVICE int32 [num_free] or NULL; only the
 * number of requests is a host value.  Needs fixed launches (as_plan_set_fixed_launch), so the whole step - this
 * call, as_verify_attn per layer, as_accept, as_kv_commit - can be recorded once in a CUDA graph and replayed step
 * after step with nothing read back by the host (Sec. 4.2 / Eq. 3: the draft lengths change from step to step, the
 * recording does not).  The work list is the one as_plan() builds for the same lengths, entry
 * for entry (both use one cost model and one cutting rule).  What as_plan() rejects with an error code cannot be
 * reported that way here: lengths out of range, a request that needs more pages than max_blocks_per_req, more
 * rows or pages than the plan's capacity, or a free list that is too short raise AS_FLAG_BAD_PLAN in the status
 * word (as_plan_check) and leave an EMPTY step behind, so the following calls do nothing.  Free page ids are not
 * range-checked here; a bad one raises AS_FLAG_BAD_PAGE where it is used.  as_plan_stats() reports -1 items. */
AS_API int as_plan_device(as_plan_t* plan, int batch, const int32_t* seq_lens, const int32_t* draft_lens,
                   int32_t* block_table, const int32_t* free_blocks, int num_free, void* stream);

/* Verify attention for layer flavour `kind` (reading: Sec. 2.2 says no more than that the target
 * model verifies the drafts; the mask is the causal chain that a single drafted continuation implies, Sec. 4.2).
 *   q: dev bf16 [total_q, Hq, D].  k_new, v_new: dev bf16 [total_q, Hkv, D], the K/V of the step's
 *   own tokens.  k_pool, v_pool: dev bf16 [num_blocks, Hkv, bs, D] (16-byte aligned), updated in
 *   place: row j of request i is first stored at position n_i + j (tentative append), then
 *   out[cu_q[i]+j, h, :] = softmax_t(sm_scale * <q, K_t>) V_t over t in [lo, n_i+j], lo = 0 or
 *   max(0, n_i+j-W+1), with kv-head h / G, plus the sink term in the denominator if the kind has one.
 *   out: dev bf16 [total_q, Hq, D].  lse: dev fp32 [total_q, Hq] natural-log normaliser, or NULL.
 * block_table must be the one given to as_plan().  Products are bf16 x bf16 accumulated in fp32;
 * softmax weights are rounded to bf16 before the PV product. */
AS_API int as_verify_attn(as_plan_t* plan, int kind, const void* q, const void* k_new, const void* v_new, void* k_pool,
                   void* v_pool, const int32_t* block_table, void* out, float* lse, void* stream);

/* Acceptance over the vocabulary (reading of lossless verification, Sec. 2.2; rejection rate of
 * Sec. 3 = 1 - sum a_i / sum k_i).  Logit row j of request i judges draft j+1.
 *   logits: dev fp32 [total_q, ld], ld >= vocab.  draft_tokens: dev int32 [total_d].
 *   temperature: dev fp32 [batch] or NULL.  NULL or T_i <= 0: greedy, the draft must equal the
 *     lowest-index maximum of its row (NaN never wins; a row with nothing comparable gives 0).
 *   T_i > 0: p = softmax(z / T_i); accept while u < min(1, p[d] / q[d]); q = draft_probs row
 *     (dev fp32 [total_d, ld]) or, if draft_probs is NULL, one-hot at the draft (model-free drafter,
 *     the paper's case).  u: dev fp32 [total_d] in [0,1), one per draft; w: dev fp32 [total_q], one
 *     per row, of which only row a_i is used: the extra token is the inverse CDF at w of
 *     max(0, p - q) after a rejection, of p after a full accept (strict '>', so zero-mass tokens are
 *     never chosen).  u and w may be NULL when no request samples.
 *   accept_len: dev int32 [batch] <- a_i.  out_tokens: dev int32 [batch, max_draft + 1] <- the a_i
 *   accepted drafts, then the extra token, then -1 padding. */
AS_API int as_accept(as_plan_t* plan, const float* logits, int64_t ld, int vocab, const int32_t* draft_tokens,
              const float* draft_probs, const float* temperature, const float* u, const float* w,
              int32_t* accept_len, int32_t* out_tokens, void* stream);

/* as_accept() for sampling requests with the uniforms drawn inside the kernels instead of passed in, so that
 * a step needs no host-made random numbers.  rng_state: dev uint64 [2] = {seed, step}, read when the kernels
 * run (the caller advances `step` between steps, e.g. with a small copy on the stream; the library never
 * writes it).  Generator: Philox4x32-10 (counter-based, Salmon et al., SC 2011).  Block (i, b) has counter
 * (i, b, step low, step high) and key (seed low, seed high), i = index of the request in this step's batch;
 * draft j (0-based) of request i uses word j mod 4 of block (i, j / 4) as u, the extra token uses word 0
 * of block (i, 2^31) as w; a word x becomes the float (x >> 8) * 2^-24.  Everything else as as_accept();
 * temperature must be given (requests with T_i <= 0 are still greedy).  The paper does not say where
 * its verifier's random numbers come from. */
AS_API int as_accept_seeded(as_plan_t* plan, const float* logits, int64_t ld, int vocab, const int32_t* draft_tokens,
                            const float* draft_probs, const float* temperature, const uint64_t* rng_state,
                            int32_t* accept_len, int32_t* out_tokens, void* stream);

/* Greedy acceptance straight from the target model's final hidden states: the output projection
 *   logits[r][v] = sum_h hidden[r][h] * weight[v][h]
 * is computed on the tensor cores tile by tile and every tile is reduced at once to the row's largest logit and its
 * lowest column, so the [total_q, vocab] logits are never written to memory; the decision is then as_accept()'s
 * greedy one (reading: Sec. 2.2 says only that the target model verifies the drafts; the paper's Sec. 3 names the growth of the
 * verification cost with the number of drafted tokens, which at large batches is this projection).
 *   hidden: dev bf16 [rows, hidden_dim], row stride hidden_dim, row r = row r of as_accept's logits; it must hold
 *     total_q rows (with fixed launches: max_batch * (max_draft + 1) rows, readable, contents beyond total_q unused).
 *   weight: dev bf16 [vocab, hidden_dim] (one row per vocabulary entry).  hidden_dim a multiple of 64; both 16-byte aligned.
 * Products are bf16 x bf16 accumulated in fp32 by the tensor cores in their own order, so against an exact evaluation
 * the argmax of a row can differ where the two largest logits are closer than that accumulation error; -0 = +0,
 * NaN counts as -inf, ties go to the lowest column, as in as_accept().  Sampling requests need the logits
 * themselves and are not served by this call. */
AS_API int as_accept_lm_head(as_plan_t* plan, const void* hidden, const void* weight, int hidden_dim, int vocab,
                      const int32_t* draft_tokens, int32_t* accept_len, int32_t* out_tokens, void* stream);

/* The same fusion for sampling requests (lossless rejection sampling, the reading of as_accept): the projection
 * is computed tile by tile and reduced at once to what the accept test needs of a row - its argmax, the online pair
 * (max, sum of exp((z - max) / T)) and the single logit z[d] of the row's draft token - so that p[d] is known without
 * any logits in memory; the extra token is then drawn from the recovery distribution of ONE row per request (row a_i),
 * whose logits a second, small pass over the weights writes to `scratch` (batch rows instead of total_q).
 *   hidden, weight, hidden_dim, vocab, draft_tokens, accept_len, out_tokens: as for as_accept_lm_head.
 *   draft_probs: dev fp32 [total_d, ld] (ld >= vocab) or NULL for a one-hot drafter; temperature: dev fp32 [batch],
 *     required (T_i <= 0 = greedy for that request); u, w: dev fp32 [total_d], [total_q]; or rng_state: dev uint64 [2]
 *     {seed, step} for uniforms drawn in the kernels exactly as as_accept_seeded draws them (then u, w may be NULL).
 *   scratch: dev, 256-byte aligned, at least as_accept_lm_head_scratch_bytes(plan, hidden_dim, vocab) bytes (sized
 *     for the plan's maxima); contents are scratch.
 * Decisions equal as_accept's on the logits hidden x weight^T except where a ratio min(1, p/q) lies within the
 * projection's accumulation error of its uniform (the tensor cores sum bf16 products in fp32, in their own order). */
AS_API size_t as_accept_lm_head_scratch_bytes(const as_plan_t* plan, int hidden_dim, int vocab);
AS_API int as_accept_lm_head_sampled(as_plan_t* plan, const void* hidden, const void* weight, int hidden_dim, int vocab,
                                     const int32_t* draft_tokens, const float* draft_probs, int64_t ld,
                                     const float* temperature, const float* u, const float* w, const uint64_t* rng_state,
                                     void* scratch, size_t scratch_bytes, int32_t* accept_len, int32_t* out_tokens,
                                     void* stream);

/* Commit / rollback (paper: silent; this is the bookkeeping any paged cache needs after a verify
 * step).  seq_lens: dev int32 [batch], in: n_i, out: n_i + a_i + 1.  Every page of request i with
 * logical index >= ceil(n_i'/bs) that the step held is released: its table entry becomes -1 and
 * its id is appended to freed[] in (request, logical page) order; *freed_count receives the
 * total.  freed: dev int32 [batch * (max_draft/bs + 2)].  With AS_COMMIT_SCRUB, k_pool / v_pool
 * (may be NULL otherwise) get zeros in the rejected slots of pages that stay held; without it
 * those bytes are unspecified and never read again. */
AS_API int as_kv_commit(as_plan_t* plan, const int32_t* accept_len, int32_t* seq_lens, int32_t* block_table,
                 int32_t* freed, int32_t* freed_count, int flags, void* k_pool, void* v_pool, void* stream);

/* Synchronises `stream`, reads the status word and clears it.  AS_OK, AS_ERR_DEVICE_FLAG or
 * AS_ERR_TIMEOUT; *flags (host, may be NULL) receives the AS_FLAG_* bits. */
AS_API int as_plan_check(as_plan_t* plan, uint32_t* flags, void* stream);

/* Introspection for tests and the benchmark: number of CTAs the attention kernel of `kind` is
 * launched with, work items and merged pairs of the current step, and which kernel runs
 * (AS_ATTN_SIMT / AS_ATTN_TC).  Any out pointer may be NULL. */
AS_API int as_plan_stats(const as_plan_t* plan, int kind, int* num_ctas, int* num_items, int* num_merges, int* impl);

/* Timing hook for benchmarks: when both are non-NULL (cudaEvent_t handles passed as void*), every
 * following as_verify_attn() records `begin` on the stream just before its main attention kernel
 * and `end` just after it (the append and merge kernels fall outside the pair).  NULL, NULL turns
 * the hook off.  The events stay owned by the caller. */
AS_API int as_plan_set_profile_events(as_plan_t* plan, void* begin, void* end);
/* Number of kernels this plan has launched since it was created (all calls, all streams). */
AS_API int64_t as_plan_launch_count(const as_plan_t* plan);

/* Test hook (no counterpart in the paper): exercises the bounded waits of the tensor-core attention kernels without
 * any fault.  Every wait inside those kernels gives up after a time limit (2 s), raises AS_FLAG_WAIT_CAP plus a bit
 * that names the wait, lets the CTA's other roles leave their loops, waits for copies in flight, frees its tensor
 * memory and returns; as_plan_check() then reports AS_ERR_TIMEOUT.  This call shortens the limit to wait_limit_ns
 * (0 = the default) and makes every CTA's copy producers stop issuing after stall_after_loads tile copies (-1 =
 * never), so that the waits behind them run out.  The attention output of such a step is unspecified; nothing is
 * read or written out of range, and the plan, the workspace and the device stay usable.  Applies to the following
 * as_verify_attn calls of this plan until reset with (0, -1). */
AS_API int as_plan_set_test_stall(as_plan_t* plan, uint64_t wait_limit_ns, int stall_after_loads);

/* Greedy acceptance for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this is a convenience of the library, not part of the method.)
 *
 * Who needs it: code that runs where no allocation call is permitted - a serving process whose
 * device memory belongs entirely to its framework's pool and that may not call cudaMalloc behind
 * the pool's back, or a latency-critical loop in which an allocating call (and the synchronisation
 * it implies) is forbidden.  as_accept() needs a caller-provided workspace for its per-row partial
 * results; this entry point keeps them in a fixed array inside the library's device image instead, so
 * the caller passes only inputs and outputs.  It calls no cudaMalloc / cudaFree and no routine that
 * allocates.  The price: every GPU that loads the library holds that array (about 0.5 MB) until the
 * process exits, and one call handles at most AS_STATIC_MAX_ROWS query rows (sum of k_i + 1); more
 * rows -> AS_ERR_INVALID_ARG with a message naming the limit.
 *
 *   batch requests, total_q = sum (k_i + 1) rows, every k_i <= max_draft.
 *   cu_q: dev int32 [batch + 1], first row of each request (cu_q[batch] = total_q); k_i is
 *     cu_q[i+1] - cu_q[i] - 1 and request i's drafts start at draft_tokens[cu_q[i] - i].
 *   logits: dev fp32 [total_q, ld], ld >= vocab.  draft_tokens: dev int32 [total_q - batch].
 *   accept_len: dev int32 [batch]; out_tokens: dev int32 [batch, max_draft + 1] (-1 padded).
 * Same rule and same results as as_accept() with temperature = NULL: a draft is accepted while it
 * equals the lowest-index maximum of its row (NaN never wins), then the extra token follows.
 * cu_q is read on the device and is not trusted: a request whose entries do not describe between 0 and
 * max_draft drafts inside rows [0, total_q) gets accept_len 0 and a row of -1 (this entry point has no
 * status word to report it through); the other requests are unaffected and nothing is read out of range.
 * Work is enqueued on `stream` for the current device.  The first call on a device looks up the
 * array's device address (cudaGetSymbolAddress, with that device current); make that first call
 * outside any stream capture.  All calls on a device share the one array and it keeps the previous
 * call's contents (the call clears the part that must start at zero), so two calls whose kernels
 * may overlap on the GPU - different streams without an ordering between them - race with each other. */
#define AS_STATIC_MAX_ROWS 1024
AS_API int as_accept_greedy_static(int batch, int total_q, int max_draft, const int32_t* cu_q, const float* logits,
                                   int64_t ld, int vocab, const int32_t* draft_tokens, int32_t* accept_len,
                                   int32_t* out_tokens, void* stream);

/* Redundancy-aware budget allocation (Sec. 4.2, Eq. 1-3; Algorithm 2): the draft lengths that as_plan()
 * consumes.  Host-only, no device access, no plan needed; every pointer is a host pointer.
 *   num_candidates[i] = n_i: continuations retrieved from the history for request i (>= 0);
 *   agree_count[i]    = c_i: how many of them agree on the most frequent prefix (0 <= c_i <= n_i);
 *   prefix_len[i]     = |CT_i|: length of that prefix in tokens (>= 0);
 *   alpha >= 0: overall speculative budget; 0 <= g_min <= 1: confidence under low support.
 * Computes g_i = c_i/n_i * (g_min + (1 - g_min)(1 - e^(1 - n_i))) (0 when n_i = 0; the exponent of the
 * body of Sec. 4.2, so that one candidate gives exactly g_min), B_t = floor(alpha / batch) and
 * draft_lens[i] = max(prefix_len[i], floor(B_t * g_i / sum_j g_j)); when all scores are 0 every request
 * keeps prefix_len[i].  Scores are summed in request order in fp64.  max_len > 0 additionally caps
 * every length (the plan's max_draft; the paper has no cap), 0 = no cap.  scores (may be NULL)
 * receives g_i.  AS_ERR_INVALID_ARG on a null pointer or a value outside the ranges above. */
AS_API int as_budget(int batch, const int32_t* agree_count, const int32_t* num_candidates, const int32_t* prefix_len,
                     double alpha, double g_min, int max_len, int32_t* draft_lens, double* scores);

/* Host-only preview of the split-KV work list as_plan() would build for `kind` with num_ctas
 * shares (0 = the count the selected kernel uses) if all requests went into one launch (no bucketing by
 * row count): no device access, nothing is stored in the plan.  items: host int32 [cap_items, 5] <- (request, kv_head, key_begin, key_end, part_row) per
 * item in CTA order; cta_first: host int32 [num_ctas + 1].  *num_items receives the item count
 * (items beyond cap_items are not written).  For tests of the planner. */
AS_API int as_plan_preview(const as_plan_t* plan, int kind, int num_ctas, int batch, const int32_t* seq_lens,
                    const int32_t* draft_lens, int32_t* items, int cap_items, int32_t* cta_first, int* num_items,
                    int* num_ctas_out);

/* Structure-isolated drafting (Sec. 4.1, Algorithm 1): host-only, no device access, no plan needed.
 * The paper fixes the structure - a cached token-to-string map M, a string pushdown automaton over the start / end
 * tags of the semantic blocks B_i, one history cache per (agent a_i, query q_i, block), drafts retrieved from the
 * matched block only - and leaves the details open; the readings taken are:
 *   - the text of a request is the concatenation of its tokens' strings (bytes); tags are recognised left to right
 *     and never overlap: after each byte, if the bytes since the previous tag end with the end tag of the innermost
 *     open block that block is closed, otherwise the first block in list order whose start tag they end with is
 *     opened (blocks nest; an end tag of a block that is not innermost is plain text);
 *   - a token belongs to the innermost open block after its last byte (-1: none); the history of (agent, query,
 *     block) is the list, in order of creation, of the maximal runs of consecutive tokens of one request that belong
 *     to the block; it outlives the requests that wrote it;
 *   - the context of a request is the last min(match_len, length of its current run) tokens of that run; every
 *     place in the same (agent, query, block) history where the context is followed by at least one token yields a
 *     candidate continuation of up to max_len tokens (the request's own run takes part);
 *   - the most frequent continuation prefix CT: its first token is the most frequent first token of the candidates
 *     (ties: the smallest id); it grows while more than half of the candidates that still agree with it continue
 *     with the same token, up to max_len tokens.
 * as_drafter_create: token_strings[t] / token_bytes[t] = the bytes of token t (may be empty), copied.
 * as_drafter_open: a request of (agent, query) whose blocks are the num_blocks (start, end) pairs of non-empty
 *   NUL-terminated tags; *request receives its handle.  as_drafter_close ends it (its history stays).
 * as_drafter_forget: drops every history of (agent, query) - the caller's way to bound memory once a query is
 *   finished; AS_ERR_INVALID_ARG while one of its requests is still open.
 * as_drafter_feed: the request's newly generated tokens, in order.  as_drafter_block: block of its last token, -1
 *   outside every block (-2: no such request).
 * as_drafter_propose: prefix (room for max_len ids) receives CT, *prefix_len = |CT|, *num_candidates = n,
 *   *agree_count = c = candidates that have CT as a prefix: exactly the three inputs of as_budget() for this
 *   request; all zero when the request is outside every block or nothing matches. */
typedef struct as_drafter_s as_drafter_t;
AS_API int as_drafter_create(as_drafter_t** out, const char* const* token_strings, const int32_t* token_bytes, int vocab);
AS_API int as_drafter_destroy(as_drafter_t* drafter);
AS_API int as_drafter_open(as_drafter_t* drafter, int64_t agent, int64_t query, const char* const* start_tags,
                    const char* const* end_tags, int num_blocks, int* request);
AS_API int as_drafter_close(as_drafter_t* drafter, int request);
AS_API int as_drafter_forget(as_drafter_t* drafter, int64_t agent, int64_t query);
AS_API int as_drafter_feed(as_drafter_t* drafter, int request, const int32_t* tokens, int n);
AS_API int as_drafter_block(const as_drafter_t* drafter, int request);
AS_API int as_drafter_propose(as_drafter_t* drafter, int request, int match_len, int max_len, int32_t* prefix, int* prefix_len,
                       int* num_candidates, int* agree_count);

#ifdef __cplusplus
}
#endif
#endif /* AS_VERIFY_H_ */
