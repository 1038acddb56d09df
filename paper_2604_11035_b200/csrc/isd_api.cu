// Host side of the C ABI: configuration checks, scratch ownership, launch sequencing.
#include <math.h>
#include <new>
#include <stdio.h>

#include "isd_internal.cuh"

int isd_attn_tc_create(isd_ctx* ctx);
void isd_attn_tc_destroy(isd_ctx* ctx);

// CTAs per row of the verification's first pass and pieces per sampled row of its second (isd_verify.cu)
int isd_pick_row_splits(const isd_config& c, int num_sms);
int isd_pick_sample_splits(const isd_config& c, int num_sms);

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <typename T>
int dev_alloc(T** p, size_t n) {
  *p = nullptr;
  if (n == 0) n = 1;
  return cudaMalloc(reinterpret_cast<void**>(p), n * sizeof(T)) == cudaSuccess ? ISD_OK : ISD_ERR_NO_MEMORY;
}

int check_state(const isd_batch_state* st) {
  if (!st) return ISD_ERR_INVALID_ARG;
  if (!st->ctx_len || !st->n_ver || !st->block_tok || !st->q_row0 || !st->page_table || !st->free_stack ||
      !st->free_top || !st->active || !st->slot_status)
    return ISD_ERR_INVALID_ARG;
  return ISD_OK;
}

int check_out(const isd_ctx* ctx, const isd_verify_out* o) {
  if (!o) return ISD_ERR_INVALID_ARG;
  if (!o->accept_len || !o->n_emit || !o->repl_tok || !o->out_tok) return ISD_ERR_INVALID_ARG;
  if (ctx->cfg.stride > 1 && (!o->accept || !o->alpha || !o->new_prop_tok || !o->new_q_stats))
    return ISD_ERR_INVALID_ARG;
  return ISD_OK;
}

}  // namespace

extern "C" {

int isd_create(const isd_config* cfg, isd_ctx** out) {
  if (!cfg || !out) return ISD_ERR_INVALID_ARG;
  *out = nullptr;
  const isd_config& c = *cfg;
  if (c.batch < 1 || c.batch > 65535 || c.stride < 1 || c.n_q_heads < 1 || c.n_kv_heads < 1 || c.vocab < 8 ||
      c.max_pages_per_slot < 1 || c.num_pages < 1 || c.n_q_heads % c.n_kv_heads != 0)
    return ISD_ERR_INVALID_ARG;
  if (c.logits_dtype != ISD_LOGITS_F32 && c.logits_dtype != ISD_LOGITS_BF16) return ISD_ERR_INVALID_ARG;
  if (c.q_mode < 0 || c.q_mode > 1 || c.propose_mode < 0 || c.propose_mode > 1) return ISD_ERR_INVALID_ARG;
  if (!(c.inv_temperature > 0.f) || !(c.tau >= 0.f)) return ISD_ERR_INVALID_ARG;
  if (c.top_k < 0 || (c.top_k > 0 && !(c.top_p > 0.f && c.top_p <= 1.f))) return ISD_ERR_INVALID_ARG;
  if (c.top_k > ISD_MAX_TOP_K) return ISD_ERR_UNSUPPORTED;
  const int Q = 2 * c.stride - 1;
  const int G = c.n_q_heads / c.n_kv_heads;
  if (c.head_dim != ISD_HEAD_DIM || c.page_size != ISD_PAGE || Q > ISD_MAX_Q || G * Q > 128 || c.vocab % 8 != 0)
    return ISD_ERR_UNSUPPORTED;

  isd_ctx* ctx = new (std::nothrow) isd_ctx();
  if (!ctx) return ISD_ERR_NO_MEMORY;
  ctx->cfg = c;
  ctx->Q = Q;
  ctx->G = G;
  ctx->sm_scale = c.sm_scale > 0.f ? c.sm_scale : 1.0f / sqrtf((float)c.head_dim);
  ctx->launches = 0;
  ctx->wait_ns = ISD_DEFAULT_WAIT_NS;
  if (cudaGetDevice(&ctx->device) != cudaSuccess) { delete ctx; return ISD_ERR_CUDA; }
  int sms = 0;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, ctx->device);
  ctx->num_sms = sms > 0 ? sms : ISD_NUM_SMS_DEFAULT;

  const int rows = c.batch * Q;
  const int rs = isd_pick_row_splits(c, ctx->num_sms);
  ctx->row_splits = rs;
  // every slot samples one row (bonus token or residual replacement; N rows with sampled proposals)
  // in the second pass
  const int ps = isd_pick_sample_splits(c, ctx->num_sms);
  ctx->sample_splits = ps;

  int rc = ISD_OK;
  if (rc == ISD_OK) rc = dev_alloc(&ctx->row_part, (size_t)rows * rs * 8);  // one partial per worker warp of a row piece
  if (rc == ISD_OK) rc = dev_alloc(&ctx->samp_part, (size_t)c.batch * c.stride * ps);
  if (rc == ISD_OK) rc = dev_alloc(&ctx->samp_ticket, (size_t)c.batch * c.stride);
  if (rc == ISD_OK) rc = dev_alloc(&ctx->global_status, 1);
  if (rc == ISD_OK) rc = dev_alloc(&ctx->step_ticket, 1);
  if (rc == ISD_OK) {
    cudaMemset(ctx->step_ticket, 0, sizeof(int));
    cudaMemset(ctx->samp_ticket, 0, sizeof(int) * c.batch * c.stride);
    cudaMemset(ctx->global_status, 0, sizeof(uint32_t));
  }
  if (rc == ISD_OK && c.top_k > 0) rc = isd_verify_topk_create(ctx);
  if (rc == ISD_OK) rc = isd_lora_create(ctx);
  if (rc == ISD_OK) rc = isd_attn_tc_create(ctx);
  if (rc == ISD_OK && cudaDeviceSynchronize() != cudaSuccess) rc = ISD_ERR_CUDA;
  if (rc != ISD_OK) {
    isd_destroy(ctx);
    return rc;
  }
  *out = ctx;
  return ISD_OK;
}

int isd_destroy(isd_ctx* ctx) {
  if (!ctx) return ISD_ERR_INVALID_ARG;
  cudaDeviceSynchronize();
  isd_attn_tc_destroy(ctx);
  isd_verify_topk_destroy(ctx);
  isd_lora_destroy(ctx);
  cudaFree(ctx->row_part);
  cudaFree(ctx->samp_part);
  cudaFree(ctx->samp_ticket);
  cudaFree(ctx->global_status);
  cudaFree(ctx->step_ticket);
  delete ctx;
  return ISD_OK;
}

int isd_attn(isd_ctx* ctx, const isd_batch_state* st, const void* q, const void* k_new, const void* v_new,
             void* k_pool, void* v_pool, void* attn_out, float* attn_lse, void* cuda_stream) {
  if (!ctx) return ISD_ERR_INVALID_ARG;
  int rc = check_state(st);
  if (rc != ISD_OK) return rc;
  if (!q || !k_new || !v_new || !k_pool || !v_pool || !attn_out) return ISD_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(k_pool) || !aligned16(v_pool) ||
      !aligned16(attn_out))
    return ISD_ERR_ALIGNMENT;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  rc = isd_launch_kv_append(ctx, st, k_new, v_new, k_pool, v_pool, s);
  if (rc != ISD_OK) return rc;
  return isd_launch_attn_tc(ctx, st, q, k_new, v_new, k_pool, v_pool, attn_out, attn_lse, s);
}

int isd_verify(isd_ctx* ctx, const isd_batch_state* st, const void* logits_cur, const void* q_prev_logits,
               uint64_t step, const isd_verify_out* out, void* cuda_stream) {
  if (!ctx) return ISD_ERR_INVALID_ARG;
  int rc = check_state(st);
  if (rc != ISD_OK) return rc;
  rc = check_out(ctx, out);
  if (rc != ISD_OK) return rc;
  if (!logits_cur || step > 0xFFFFFFFFull) return ISD_ERR_INVALID_ARG;
  if (ctx->cfg.stride > 1 && !st->q_stats) return ISD_ERR_INVALID_ARG;
  if (!aligned16(logits_cur) || (q_prev_logits && !aligned16(q_prev_logits))) return ISD_ERR_ALIGNMENT;
  if (ctx->cfg.top_k > 0)
    return isd_launch_verify_topk(ctx, st, logits_cur, q_prev_logits, (uint32_t)step, out,
                                  reinterpret_cast<cudaStream_t>(cuda_stream));
  return isd_launch_verify(ctx, st, logits_cur, q_prev_logits, (uint32_t)step, out,
                           reinterpret_cast<cudaStream_t>(cuda_stream));
}

int isd_commit(isd_ctx* ctx, isd_batch_state* st, const isd_verify_out* out, void* cuda_stream) {
  if (!ctx) return ISD_ERR_INVALID_ARG;
  int rc = check_state(st);
  if (rc != ISD_OK) return rc;
  rc = check_out(ctx, out);
  if (rc != ISD_OK) return rc;
  return isd_launch_commit(ctx, st, out, reinterpret_cast<cudaStream_t>(cuda_stream));
}

// Verification followed by the commit: the last CTA of the last verification kernel commits (no kernel of its
// own for it), except on the filtered path when the proposal-law rows have to be streamed by a second kernel.
static int verify_then_commit(isd_ctx* ctx, isd_batch_state* st, const void* logits_cur, const void* q_prev_logits,
                              uint64_t step, const isd_verify_out* out, void* cuda_stream) {
  int rc = check_state(st);
  if (rc != ISD_OK) return rc;
  rc = check_out(ctx, out);
  if (rc != ISD_OK) return rc;
  if (!logits_cur || step > 0xFFFFFFFFull) return ISD_ERR_INVALID_ARG;
  if (ctx->cfg.stride > 1 && !st->q_stats) return ISD_ERR_INVALID_ARG;
  if (!aligned16(logits_cur) || (q_prev_logits && !aligned16(q_prev_logits))) return ISD_ERR_ALIGNMENT;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (ctx->cfg.top_k > 0) {
    bool committed = false;
    rc = isd_launch_verify_topk(ctx, st, logits_cur, q_prev_logits, (uint32_t)step, out, s, st, &committed);
    if (rc != ISD_OK || committed) return rc;
    return isd_launch_commit(ctx, st, out, s);
  }
  return isd_launch_verify(ctx, st, logits_cur, q_prev_logits, (uint32_t)step, out, s, st);
}

int isd_step(isd_ctx* ctx, isd_batch_state* st, const isd_step_args* a, uint64_t step, void* cuda_stream) {
  if (!ctx || !a) return ISD_ERR_INVALID_ARG;
  int rc = isd_attn(ctx, st, a->q, a->k_new, a->v_new, a->k_pool, a->v_pool, a->attn_out, a->attn_lse, cuda_stream);
  if (rc != ISD_OK) return rc;
  return verify_then_commit(ctx, st, a->logits_cur, a->q_prev_logits, step, &a->out, cuda_stream);
}

int isd_step_layers(isd_ctx* ctx, isd_batch_state* st, const isd_layer_args* layers, int32_t n_layers,
                    const void* logits_cur, const void* q_prev_logits, const isd_verify_out* out, uint64_t step,
                    void* cuda_stream) {
  if (!ctx || !layers || n_layers < 1 || !out) return ISD_ERR_INVALID_ARG;
  // every layer attends through the same page table and lengths: the state changes only in the commit
  for (int32_t l = 0; l < n_layers; ++l) {
    const isd_layer_args& a = layers[l];
    const int rc = isd_attn(ctx, st, a.q, a.k_new, a.v_new, a.k_pool, a.v_pool, a.attn_out, a.attn_lse, cuda_stream);
    if (rc != ISD_OK) return rc;
  }
  return verify_then_commit(ctx, st, logits_cur, q_prev_logits, step, out, cuda_stream);
}

int isd_lora_linear(isd_ctx* ctx, const isd_lora_args* a, void* cuda_stream) {
  if (!ctx || !a || !a->x || !a->w || !a->a || !a->b || !a->gate || !a->t || !a->y) return ISD_ERR_INVALID_ARG;
  if (a->m < 1 || a->n < 1 || a->k < 1 || a->rank < 1) return ISD_ERR_INVALID_ARG;
  if (a->k % 64 != 0 || a->rank % 64 != 0 || a->n % 32 != 0) return ISD_ERR_UNSUPPORTED;
  if (!aligned16(a->x) || !aligned16(a->w) || !aligned16(a->a) || !aligned16(a->b) || !aligned16(a->t) || !aligned16(a->y))
    return ISD_ERR_ALIGNMENT;
  return isd_launch_lora_linear(ctx, a, reinterpret_cast<cudaStream_t>(cuda_stream));
}

int isd_set_wait_limit(isd_ctx* ctx, uint32_t milliseconds) {
  if (!ctx || milliseconds == 0) return ISD_ERR_INVALID_ARG;
  ctx->wait_ns = (unsigned long long)milliseconds * 1000000ull;
  return ISD_OK;
}

int isd_test_preset_lora_counter(isd_ctx* ctx, int32_t row_block, uint32_t value, void* cuda_stream) {
  if (!ctx || !ctx->lora_flags || row_block < 0 || row_block >= 4096) return ISD_ERR_INVALID_ARG;
  // (pageable host source: the runtime stages the four bytes before it returns)
  return cudaMemcpyAsync(ctx->lora_flags + row_block, &value, sizeof(uint32_t), cudaMemcpyHostToDevice,
                         reinterpret_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? ISD_OK : ISD_ERR_CUDA;
}

int isd_set_step_counter(isd_ctx* ctx, uint32_t* device_counter) {
  if (!ctx) return ISD_ERR_INVALID_ARG;
  ctx->step_counter = device_counter;
  return ISD_OK;
}

int isd_release(isd_ctx* ctx, isd_batch_state* st, const int32_t* slots, int32_t n, void* cuda_stream) {
  if (!ctx || !slots || n < 0) return ISD_ERR_INVALID_ARG;
  int rc = check_state(st);
  if (rc != ISD_OK) return rc;
  return isd_launch_release(ctx, st, slots, n, reinterpret_cast<cudaStream_t>(cuda_stream));
}

int isd_read_status(isd_ctx* ctx, uint32_t* host_status, void* cuda_stream) {
  if (!ctx || !host_status) return ISD_ERR_INVALID_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(host_status, ctx->global_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return ISD_ERR_CUDA;
  if (cudaMemsetAsync(ctx->global_status, 0, sizeof(uint32_t), s) != cudaSuccess) return ISD_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return ISD_ERR_CUDA;
  return ISD_OK;
}

int isd_set_profile_events(isd_ctx* ctx, void* attn_start, void* attn_stop, void* verify_start, void* verify_stop) {
  if (!ctx) return ISD_ERR_INVALID_ARG;
  ctx->ev_attn0 = reinterpret_cast<cudaEvent_t>(attn_start);
  ctx->ev_attn1 = reinterpret_cast<cudaEvent_t>(attn_stop);
  ctx->ev_verify0 = reinterpret_cast<cudaEvent_t>(verify_start);
  ctx->ev_verify1 = reinterpret_cast<cudaEvent_t>(verify_stop);
  return ISD_OK;
}

int64_t isd_launch_count(const isd_ctx* ctx) { return ctx ? ctx->launches : 0; }

const char* isd_strerror(int code) {
  switch (code) {
    case ISD_OK: return "ok";
    case ISD_ERR_INVALID_ARG: return "invalid argument";
    case ISD_ERR_UNSUPPORTED: return "unsupported configuration (head_dim must be 128, page_size 16, (Hq/Hkv)*(2N-1) <= 128, vocab % 8 == 0, top_k <= 64; isd_verify_static: top_k = 0)";
    case ISD_ERR_CUDA: return "CUDA runtime error";
    case ISD_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
    case ISD_ERR_NO_MEMORY: return "out of memory";
    case ISD_ERR_TOO_LARGE: return "batch exceeds ISD_STATIC_MAX_BATCH, the capacity of the static scratch of isd_verify_static";
    default: return "unknown error";
  }
}

}  // extern "C"
