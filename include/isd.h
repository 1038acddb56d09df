/*
 * isd.h -- C ABI of the B200 (sm_100a) introspective strided decoding (ISD) step.
 *
 * One ISD step (paper "Introspective Diffusion Language Models", Algorithm 1 in
 * its fused 2N-1 row form, Sec. 3.2 / Sec. 3.3) for a stationary batch of B slots:
 *
 *   isd_attn    strict-causal attention of every slot's query block against its
 *               paged bf16 KV cache, after appending the block's own K/V rows
 *   isd_verify  vocab-wide softmax statistics, p/q introspective acceptance,
 *               residual resample / bonus token, and the next proposals
 *   isd_commit  KV commit / rollback (keep accepted rows, drop rejected and
 *               [MASK] rows), next block, device-side page acquisition
 *   isd_step    the three chained on one stream with no host round trip
 *
 * Conventions
 *   N  = stride;  Q = 2N-1 = rows of a query block;  G = n_q_heads / n_kv_heads.
 *   Block rows of slot b: row 0 = anchor (last finalised token, no KV yet),
 *   rows 1..n_ver[b] = proposals under verification, rows n_ver[b]+1 ..
 *   n_ver[b]+N-1 = [MASK] rows, remaining rows = padding.  q_len[b] = n_ver[b]+N.
 *   Row r sits at sequence position ctx_len[b] + r.  The logits row r predicts
 *   the token at position ctx_len[b] + r + 1 (logit shift, Sec. 3.1).
 *
 * Memory
 *   Every pointer inside the structs below and every tensor argument is a DEVICE
 *   pointer owned by the caller, 16-byte aligned, dense row-major in the stated
 *   shape.  The library allocates only its own scratch (inside isd_ctx, at
 *   isd_create) and never frees or reallocates caller memory.  State and pools
 *   are updated in place.  Pointers of type `const isd_config*`, `isd_ctx**`,
 *   the structs themselves and `host_status` are HOST pointers.
 *
 * Errors
 *   Every call returns 0 or a negative ISD_ERR_* code (argument / CUDA errors,
 *   detected on the host before anything is launched).  Data-dependent faults
 *   (bad token or page ids, exhausted pool, non-finite logits) never trap: they
 *   set ISD_ST_* bits in slot_status[b] and in a global word readable with
 *   isd_read_status; a slot with an error bit keeps its state (isd_commit skips
 *   it) so that the caller can repair it and clear the bit.
 *
 * Threading / streams
 *   Calls are asynchronous on `cuda_stream` (a cudaStream_t passed as void*),
 *   except isd_create, isd_destroy and isd_read_status, which synchronise.  One
 *   isd_ctx serves one stream at a time.
 */
#ifndef ISD_H_
#define ISD_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ISD_OK 0
#define ISD_ERR_INVALID_ARG (-1)
#define ISD_ERR_UNSUPPORTED (-2)
#define ISD_ERR_CUDA (-3)
#define ISD_ERR_ALIGNMENT (-4)
#define ISD_ERR_NO_MEMORY (-5)

/* bits of slot_status[b] and of the global status word */
#define ISD_ST_POOL_EXHAUSTED 1u  /* free stack could not serve the slot's request   */
#define ISD_ST_SLOT_CAPACITY 2u   /* slot would exceed max_pages_per_slot / bad n_ver */
#define ISD_ST_BAD_TOKEN_ID 4u    /* proposal token outside [0, vocab)                */
#define ISD_ST_BAD_PAGE_ID 8u     /* page table entry outside [0, num_pages)          */
#define ISD_ST_NONFINITE_LOGIT 16u /* NaN or +inf logit (-inf is legal)               */
#define ISD_ST_EMPTY_RESIDUAL 32u /* informational: residual max(0,p-q) was empty in
                                     fp32, token drawn from p instead; not an error  */
#define ISD_ST_KERNEL_TIMEOUT 0x80000000u /* a wait inside a kernel (on a shared-memory
                                     barrier or on another CTA's readiness counter) outlasted
                                     its time limit (isd_set_wait_limit): the CTA stopped
                                     issuing work, drained its copies, freed what it held and
                                     returned.  The results of that call are incomplete.  In
                                     the verification kernels the bit is also set in
                                     slot_status[b], so that isd_commit leaves the slot alone;
                                     the attention and LoRA kernels report it in the global
                                     word only (their CTAs serve many slots)               */

#define ISD_LOGITS_F32 0
#define ISD_LOGITS_BF16 1

typedef struct isd_ctx isd_ctx; /* opaque; owns scratch only */

#define ISD_MAX_TOP_K 64

typedef struct isd_config {
  int32_t batch;              /* B, number of fixed slots (>= 1)                      */
  int32_t stride;             /* N >= 1 (Q = 2N-1 <= 31)                              */
  int32_t n_q_heads;          /* Hq                                                   */
  int32_t n_kv_heads;         /* Hkv, divides Hq; (Hq/Hkv) * Q <= 128                 */
  int32_t head_dim;           /* must be 128                                          */
  int32_t page_size;          /* must be 16 (tokens per KV page)                      */
  int32_t vocab;              /* V, multiple of 8                                     */
  int32_t max_pages_per_slot; /* row length of page_table                             */
  int32_t num_pages;          /* pages in k_pool / v_pool                             */
  int32_t logits_dtype;       /* ISD_LOGITS_F32 or ISD_LOGITS_BF16                    */
  int32_t q_mode;             /* 0: q = softmax(proposal logits) (Algorithm 1);
                                 1: q = point mass on the proposal (argmax proposals) */
  int32_t propose_mode;       /* 0: Gumbel-max sample of the MASK row; 1: argmax
                                 (Sec. 3.3 (3))                                       */
  int32_t mask_token_id;      /* id written into [MASK] rows of the next block        */
  float sm_scale;             /* attention scale; <= 0 selects 1/sqrt(head_dim)       */
  float inv_temperature;      /* logits are multiplied by this (1.0 = paper default)  */
  float tau;                  /* relaxed acceptance: ratio * (1 + tau), Sec. 4.3      */
  uint64_t seed;              /* Philox key                                           */
  int32_t top_k;              /* 0: plain softmax laws (Algorithm 1).  1..ISD_MAX_TOP_K:
                                 every law (anchor p, proposal q, bonus, MASK rows) is
                                 first cut to its top_k tokens (value descending, lower
                                 index on ties) and then to the shortest prefix of those
                                 whose mass reaches top_p, and renormalised (the serving
                                 sampling configuration of the paper's appendix)       */
  float top_p;                /* in (0, 1]; read only when top_k > 0                  */
} isd_config;

/* Stationary-batch state (Sec. 3.3 (2)); all arrays on the device, in place. */
typedef struct isd_batch_state {
  int32_t* ctx_len;     /* [B] tokens whose KV is committed                           */
  int32_t* n_ver;       /* [B] proposals under verification this step, 0..N-1         */
  int32_t* block_tok;   /* [B, Q] token ids of the query block                        */
  int32_t* q_row0;      /* [B] row, inside the previous step's logits buffer, of the
                           law the first proposal was drawn from                      */
  float* q_stats;       /* [B, N-1, 2] {LSE(q row * invT), q row[x^] * invT} cached
                           when the proposals were made                                */
  int32_t* page_table;  /* [B, max_pages_per_slot]; a slot owns
                           ceil((ctx_len + Q) / page_size) leading entries            */
  int32_t* free_stack;  /* [num_pages] free page ids, top at free_top-1               */
  int32_t* free_top;    /* [1]                                                        */
  uint8_t* active;      /* [B] 0 = slot is skipped everywhere                         */
  uint32_t* slot_status;/* [B] sticky ISD_ST_* bits                                   */
} isd_batch_state;

/* Results of isd_verify; device arrays owned by the caller. */
typedef struct isd_verify_out {
  int8_t* accept;        /* [B, N-1] 1 accepted, 0 first rejection, -1 not evaluated  */
  float* alpha;          /* [B, N-1] min(1, (1+tau) p/q) where evaluated, else NaN    */
  int32_t* accept_len;   /* [B] a = accepted proposals, 0..n_ver                      */
  int32_t* n_emit;       /* [B] a + 1 tokens finalised                                */
  int32_t* repl_tok;     /* [B] resampled (on rejection) or bonus token               */
  int32_t* out_tok;      /* [B, N] finalised tokens (accepted proposals, then
                            repl_tok), -1 padded                                      */
  int32_t* new_prop_tok; /* [B, N-1] proposals made by this step's MASK rows; -1 where
                            a proposal of the slot was rejected: the MASK rows were
                            conditioned on tokens that are discarded, and the next
                            step is a pure stride step (Sec. 3.2, adaptive stride)   */
  float* new_q_stats;    /* [B, N-1, 2] their {LSE, logit}; NaN where none was made   */
} isd_verify_out;

/* Everything one step consumes and produces besides the state. */
typedef struct isd_step_args {
  const void* q;             /* [B, Q, Hq, D] bf16 queries (post-RoPE)                */
  const void* k_new;         /* [B, Q, Hkv, D] bf16 keys of the block rows            */
  const void* v_new;         /* [B, Q, Hkv, D] bf16 values of the block rows          */
  void* k_pool;              /* [num_pages, Hkv, page_size, D] bf16                   */
  void* v_pool;              /* same shape                                            */
  void* attn_out;            /* [B, Q, Hq, D] bf16; rows >= q_len are not written     */
  float* attn_lse;           /* [B, Q, Hq] natural-log sum of exp(scaled scores), or NULL */
  const void* logits_cur;    /* [B, Q, V] this step's logits                          */
  const void* q_prev_logits; /* [B, Q, V] previous step's logits (read only for the
                                first rejected proposal of a slot); may be NULL when
                                q_mode = 1 or no slot verifies anything                */
  isd_verify_out out;
} isd_step_args;

/*
 * Create / destroy a context for one configuration.  isd_create validates the
 * configuration (ISD_ERR_UNSUPPORTED for head_dim != 128, page_size != 16,
 * (Hq/Hkv)*Q > 128, vocab % 8 != 0), allocates scratch on the current CUDA
 * device and synchronises.  `*out` receives the context (host pointer).
 */
int isd_create(const isd_config* cfg, isd_ctx** out);
int isd_destroy(isd_ctx* ctx);

/*
 * ISD attention (Sec. 3.1 strict causal mask; Sec. 3.3 (1) single paged kernel
 * for the 2N-1 row extend).  For every active slot b, row r < q_len[b], head h:
 *   out[b,r,h,:] = softmax_j(sm_scale * q[b,r,h,:] . K_j) V_j   over keys
 *   j <= ctx_len[b] + r of KV head h / G,
 * where keys j < ctx_len[b] come from the slot's pages and keys ctx_len[b]+i are
 * row i of k_new / v_new.  Side effect: rows 0..q_len-1 of k_new / v_new are
 * written into the slot's pages at positions ctx_len[b] .. ctx_len[b]+q_len-1
 * (batched scatter of Sec. 3.3 (2)); the pages must already be owned by the slot.
 * bf16 inputs, fp32 accumulation, bf16 output.  attn_lse may be NULL.
 */
int isd_attn(isd_ctx* ctx, const isd_batch_state* st, const void* q, const void* k_new,
             const void* v_new, void* k_pool, void* v_pool, void* attn_out, float* attn_lse,
             void* cuda_stream);

/*
 * Introspective verification and proposal (Algorithm 1: introspection loop,
 * bonus branch, stride loop; Sec. 3.2 p/q rule; Sec. 3.3 (3) fused kernel with
 * online softmax and Gumbel-max correction).  For every active slot b:
 *   for j = 1..n_ver: p = softmax(logits_cur[b,j-1] * invT), q from the cached
 *   q_stats (q_mode 0) or a point mass (q_mode 1); accept proposal
 *   block_tok[b,j] iff u < min(1, (1+tau) p(x)/q(x)) with u the Philox uniform of
 *   (seed, step, b, j); at the first rejection draw the replacement from
 *   normalize(max(0, p - q)) (reads row q_row0[b]+j-1 of q_prev_logits) and stop;
 *   if nothing is rejected draw the bonus token from row n_ver.
 *   Then every MASK row m = 1..N-1 proposes from logits_cur[b, n_ver+m]
 *   (Gumbel-max sample or argmax) and caches {LSE, logit} in new_q_stats.
 * Random numbers: Philox4x32-10, key = seed, counter = (vocab_index / 4, step, b,
 * tag << 16 | position), word vocab_index % 4; tag 0 accept uniform (position j),
 * 1 replacement / bonus noise (position a+1), 2 proposal noise (position m).
 * `step` must fit 32 bits.
 * q_prev_logits must hold what the previous step's logits_cur held (the proposals were drawn from
 * its rows).  With filtered laws (top_k > 0) the context remembers the top-k lists of the previous
 * call: when q_prev_logits is the very pointer that call got as logits_cur and `step` is that call's
 * step + 1 (and no device step counter is set), the lists are reused and the rows are not read again;
 * otherwise the rows are read and selected again.
 */
int isd_verify(isd_ctx* ctx, const isd_batch_state* st, const void* logits_cur,
               const void* q_prev_logits, uint64_t step, const isd_verify_out* out,
               void* cuda_stream);

/*
 * KV commit / rollback and next-step state (Algorithm 1 "commit KV cache";
 * Sec. 3.3 (2) trim-and-commit; appendix renewal process).  For every active,
 * fault-free slot: ctx_len += accept_len + 1 (anchor and accepted rows keep
 * their KV; rejected and MASK rows are dropped by truncation); n_ver = N-1 if
 * nothing was rejected else 0; block_tok = [repl_tok, new proposals or MASK...,
 * MASK...]; q_stats = new_q_stats; q_row0 = old n_ver + 1; pages are popped from
 * the free stack (slots ascending, logical pages ascending) until the slot owns
 * ceil((ctx_len + Q) / page_size) pages.
 */
int isd_commit(isd_ctx* ctx, isd_batch_state* st, const isd_verify_out* out, void* cuda_stream);

/* isd_attn, isd_verify, isd_commit back to back on `cuda_stream` (Sec. 3.3 (2):
 * forward -> verify -> trim -> prepare without returning to the host). */
int isd_step(isd_ctx* ctx, isd_batch_state* st, const isd_step_args* args, uint64_t step,
             void* cuda_stream);

/* One transformer layer's share of a step: its queries, the block's keys / values, its KV pools and its
 * output (same shapes and meaning as the fields of isd_step_args). */
typedef struct isd_layer_args {
  const void* q;
  const void* k_new;
  const void* v_new;
  void* k_pool;
  void* v_pool;
  void* attn_out;
  float* attn_lse; /* or NULL */
} isd_layer_args;

/*
 * A whole model step (Sec. 3.3: the 2N-1 row block goes through every layer of the model in one
 * forward pass, then verify -> trim -> prepare): isd_attn for each of the n_layers layers in order,
 * all through the same state (one page table and one set of lengths shared by the layers, each
 * layer with its own pools), then isd_verify on the logits and isd_commit.  `layers` is a host array
 * of n_layers >= 1 entries; everything else as in isd_step.  No host synchronisation and no
 * allocation happen inside, so the call (like isd_step) may be recorded into a CUDA graph by stream
 * capture on `cuda_stream`; see isd_set_step_counter for the step number of a replayed graph.
 */
int isd_step_layers(isd_ctx* ctx, isd_batch_state* st, const isd_layer_args* layers, int32_t n_layers,
                    const void* logits_cur, const void* q_prev_logits, const isd_verify_out* out,
                    uint64_t step, void* cuda_stream);

/*
 * Step number for CUDA-graph replay (Sec. 3.3 (2): the captured extend graph is replayed with its
 * metadata updated in place).  The `step` argument of isd_verify / isd_step is a host value that a
 * captured graph would freeze, and every replay would draw the same random numbers.  With a
 * device counter set (device pointer to one uint32, owned by the caller, initialised by the
 * caller), isd_verify reads the step number from it and ignores its `step` argument, and
 * isd_commit adds one to it after committing, so that replay k of a captured step runs as step
 * counter0 + k.  NULL (the default) switches back to the host argument.
 */
int isd_set_step_counter(isd_ctx* ctx, uint32_t* device_counter);

/* Arguments of isd_lora_linear: device pointers, row-major bf16 matrices. */
typedef struct isd_lora_args {
  const void* x;       /* [m, k]    activations of the step's token rows (m = B * Q)          */
  const void* w;       /* [n, k]    base weight: y = x w^T                                     */
  const void* a;       /* [rank, k] LoRA down-projection                                      */
  const void* b;       /* [n, rank] LoRA up-projection                                        */
  const uint8_t* gate; /* [m]       1 = [MASK] row (LoRA residual applied), 0 = clean row     */
  void* t;             /* [m, rank] scratch of the caller: gated down-projection              */
  void* y;             /* [m, n]    output                                                    */
  int32_t m, n, k, rank;
  float scale;         /* LoRA scaling (alpha / rank)                                         */
} isd_lora_args;

/*
 * Segment-gated LoRA linear layer of the lossless R-ISD variant (Sec. 3.2, R-ISD paragraph, Eq. 5):
 *   y[j, :] = w x[j, :] + gate[j] * scale * b (a x[j, :])
 * so that clean rows are computed with the base weights alone (their verification is lossless) and
 * only [MASK] rows see the adapter.  bf16 operands, fp32 accumulation on the tensor cores, bf16
 * results; the intermediate t = gate * scale * (x a^T) is rounded to bf16 once.  Requirements
 * (else ISD_ERR_UNSUPPORTED / ISD_ERR_ALIGNMENT): k and rank multiples of 64, n a multiple of 32,
 * 16-byte aligned pointers.  One kernel on `cuda_stream` (two when rank > 256 is not a multiple of
 * 256, or when t has more 128 x 256 blocks than the GPU has SMs), no allocation, no synchronisation.
 */
int isd_lora_linear(isd_ctx* ctx, const isd_lora_args* args, void* cuda_stream);

/* Off the hot path: return the pages of finished slots (device array `slots`
 * of n ids) to the free stack and mark them inactive. */
int isd_release(isd_ctx* ctx, isd_batch_state* st, const int32_t* slots, int32_t n,
                void* cuda_stream);

/* Synchronises the stream and copies the OR of all status bits raised since the
 * last call into *host_status (host pointer), then clears the global word. */
int isd_read_status(isd_ctx* ctx, uint32_t* host_status, void* cuda_stream);

/*
 * Time limit of the waits inside the kernels (the paper has no counterpart).  Every device-side wait of the
 * library -- on a shared-memory barrier of a copy ring, on a readiness counter another CTA raises -- gives up
 * after this long (default 250 ms) and the kernel reports ISD_ST_KERNEL_TIMEOUT instead of hanging.  The
 * limit is far above anything a healthy kernel waits for; lower it on hosts that must bound how long a
 * faulty launch can hold the GPU.  milliseconds >= 1.
 */
int isd_set_wait_limit(isd_ctx* ctx, uint32_t milliseconds);

/*
 * Test hook for the wait limit (the paper has no counterpart; not for production use).  The fused LoRA layer
 * hands blocks of its intermediate t from the CTAs that compute them to the CTAs that read them through one
 * readiness counter per row block, which a reader waits on until it EQUALS the number of blocks.  This call
 * writes `value` into the counter of `row_block` (asynchronously on `cuda_stream`), so that with a value the
 * count can never reach, the readers of that row block wait until their time limit runs out: the next
 * isd_lora_linear on this context then returns normally, the rows of that block in y are incomplete, and
 * isd_read_status carries ISD_ST_KERNEL_TIMEOUT.  The kernel clears all counters when it ends, so the call
 * after that is an ordinary one again.  Nothing faults or hangs; set a short limit first (isd_set_wait_limit).
 */
int isd_test_preset_lora_counter(isd_ctx* ctx, int32_t row_block, uint32_t value, void* cuda_stream);

/*
 * Test hook, host only (the paper has no counterpart; needs no GPU): how isd_lora_linear assigns its work for a
 * shape on a GPU of num_sms SMs.  For unit `unit_index` (a CTA, or a pair of CTAs, in block-index order) of the
 * launch that writes y and its work item `item`: out[0] = kernel form (2 CTA pairs with the down-projection fused,
 * 1 one-CTA kernel fused, 0 two launches), out[1] = units of the launch, out[2] = items of this unit, out[3] = 1 for
 * a block of the intermediate t / 0 for an output tile or strip, out[4..6] = first row, first column, columns,
 * out[7..8] = rows and columns of a full tile (out[3..6] = -1 past the unit's last item).  The CPU tests use it to
 * check that every output element is computed exactly once and that the blocks of t fall to the lowest block
 * indices, whose CTAs the hardware makes resident first.
 */
int isd_test_lora_work_item(int32_t m, int32_t n, int32_t rank, int32_t num_sms, int32_t unit_index, int32_t item,
                            int32_t* out);

/*
 * Test hook, host only (the paper has no counterpart; needs no GPU): the launch shape isd_verify picks for a
 * configuration on a GPU of num_sms SMs.  out[0] = CTAs a row of the first pass is cut into, out[1] = pieces a
 * sampled row of the second pass is cut into, out[2] / out[3] = CTAs of the two launches.  Only batch, stride, vocab
 * and propose_mode of cfg are read.  Errors: ISD_ERR_INVALID_ARG.
 */
int isd_test_verify_grid(const isd_config* cfg, int32_t num_sms, int32_t* out);

/* Optional instrumentation (the paper has no counterpart): cudaEvent_t handles, passed as void*,
 * that later calls record on their stream immediately before / after the attention main kernel
 * (attn_*) and the kernels of isd_verify together (verify_*).  NULL switches a pair off.
 * The events stay owned by the caller. */
int isd_set_profile_events(isd_ctx* ctx, void* attn_start, void* attn_stop, void* verify_start,
                           void* verify_stop);

/*
 * isd_verify without any allocation (the paper has no counterpart; this serves hosts of the
 * library).  Same computation, arguments and outputs as isd_verify, but it needs no isd_ctx: the
 * scratch of the two verification kernels lives in a fixed array inside the library's device image
 * (about 0.65 MB on every GPU that loads the library, held until the process exits).
 *
 * Who needs it: callers that cannot call cudaMalloc when they verify -- an engine that has given
 * all free device memory to its own KV-cache allocator, a latency-critical thread on which
 * allocation is forbidden, or code running while the allocator is held elsewhere.  The call uses
 * no cudaMalloc / cudaFree and no allocating library routine.
 *
 * Limits and rules
 *   - cfg->batch <= ISD_STATIC_MAX_BATCH, otherwise ISD_ERR_TOO_LARGE (nothing is launched).
 *     Only the fields of cfg that verification reads matter (batch, stride, vocab, logits_dtype,
 *     q_mode, propose_mode, inv_temperature, tau, seed).
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress, with
 *     that device current) and caches it; make that first call outside any stream capture.
 *   - All calls share the one array, which keeps the previous call's contents; the counters that
 *     must start at zero are cleared on the stream at the start of every call.  Two calls that
 *     overlap on the GPU (different streams, or different host threads on one device) race on it:
 *     serialise them.
 *   - Data faults are reported in slot_status[b] only; there is no global status word to read.
 */
#define ISD_STATIC_MAX_BATCH 64
#define ISD_ERR_TOO_LARGE (-6)
int isd_verify_static(const isd_config* cfg, const isd_batch_state* st, const void* logits_cur,
                      const void* q_prev_logits, uint64_t step, const isd_verify_out* out,
                      void* cuda_stream);

/* Number of kernel launches the library has issued through this context. */
int64_t isd_launch_count(const isd_ctx* ctx);

const char* isd_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* ISD_H_ */
