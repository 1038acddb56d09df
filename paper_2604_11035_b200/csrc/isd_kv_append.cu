// K/V append: batched scatter of the block rows into the slot's pages (Sec. 3.3 (2): "KV slots are allocated
// via a single batched scatter"; Sec. 3.3 (1): the paged-only attention kernel finds the block's own keys in the
// pages).  Runs right before the attention kernel of isd_attn_tc.cu, which starts its set-up under it.
#include "isd_internal.cuh"

namespace {

struct AttnParams {
  int B, Q, N, Hq, Hkv, G, max_pages, num_pages;
  float sm_scale;
  const int32_t* ctx_len;
  const int32_t* n_ver;
  const uint8_t* active;
  const int32_t* page_table;
  uint32_t* slot_status;
  uint32_t* global_status;
  const __nv_bfloat16* q;
  const __nv_bfloat16* k_new;
  const __nv_bfloat16* v_new;
  __nv_bfloat16* k_pool;
  __nv_bfloat16* v_pool;
  __nv_bfloat16* out;
  float* lse;
};

__device__ __forceinline__ int slot_q_len(const AttnParams& P, int b) {
  if (!P.active[b]) return 0;
  const int nv = P.n_ver[b];
  if (nv < 0 || nv > P.N - 1) return 0;
  return nv + P.N;
}

// one CTA per (slot, kv head): validate the slot's page-table prefix, then scatter the block rows
__global__ void __launch_bounds__(128) kv_append_kernel(const AttnParams P) {
  const int b = blockIdx.x, g = blockIdx.y;
  pdl_wait();
  pdl_launch_dependents();
  const int ql = slot_q_len(P, b);
  if (ql == 0) return;
  const int ctx = P.ctx_len[b];
  const int pages = (ctx + ql + ISD_PAGE - 1) / ISD_PAGE;
  __shared__ int sm_bad;
  if (threadIdx.x == 0) sm_bad = 0;
  __syncthreads();
  if (ctx < 0 || pages > P.max_pages) {
    if (threadIdx.x == 0 && g == 0) {
      atomicOr(&P.slot_status[b], ISD_ST_SLOT_CAPACITY);
      atomicOr(P.global_status, ISD_ST_SLOT_CAPACITY);
    }
    return;
  }
  for (int pg = threadIdx.x; pg < pages; pg += blockDim.x) {
    const int id = P.page_table[(size_t)b * P.max_pages + pg];
    if (id < 0 || id >= P.num_pages) sm_bad = 1;
  }
  __syncthreads();
  if (sm_bad) {
    if (threadIdx.x == 0 && g == 0) {
      atomicOr(&P.slot_status[b], ISD_ST_BAD_PAGE_ID);
      atomicOr(P.global_status, ISD_ST_BAD_PAGE_ID);
    }
    return;
  }
  // each (row, K|V) of this head is 256 bytes = 16 x 16-byte vectors
  const int vecs = ql * 2 * 16;
  for (int i = threadIdx.x; i < vecs; i += blockDim.x) {
    const int v16 = i & 15;
    const int kv = (i >> 4) & 1;
    const int r = i >> 5;
    const int pos = ctx + r;
    const int page = P.page_table[(size_t)b * P.max_pages + pos / ISD_PAGE];
    const size_t src = (((size_t)b * P.Q + r) * P.Hkv + g) * ISD_HEAD_DIM;
    const size_t dst = (((size_t)page * P.Hkv + g) * ISD_PAGE + (pos % ISD_PAGE)) * ISD_HEAD_DIM;
    const uint4* s = reinterpret_cast<const uint4*>((kv ? P.v_new : P.k_new) + src) + v16;
    uint4* d = reinterpret_cast<uint4*>((kv ? P.v_pool : P.k_pool) + dst) + v16;
    *d = *s;
  }
  // Rows of the last page beyond the block are zeroed: they are never attended (masked), but the
  // tensor-core kernel multiplies them by a zero probability, which needs finite values.
  const int end = ctx + ql;
  const int tail = (ISD_PAGE - end % ISD_PAGE) % ISD_PAGE;
  const int zvecs = tail * 2 * 16;
  for (int i = threadIdx.x; i < zvecs; i += blockDim.x) {
    const int v16 = i & 15;
    const int kv = (i >> 4) & 1;
    const int pos = end + (i >> 5);
    const int page = P.page_table[(size_t)b * P.max_pages + pos / ISD_PAGE];
    const size_t dst = (((size_t)page * P.Hkv + g) * ISD_PAGE + (pos % ISD_PAGE)) * ISD_HEAD_DIM;
    reinterpret_cast<uint4*>((kv ? P.v_pool : P.k_pool) + dst)[v16] = make_uint4(0, 0, 0, 0);
  }
}

AttnParams make_params(isd_ctx* ctx, const isd_batch_state* st, const void* q, const void* k_new,
                       const void* v_new, void* k_pool, void* v_pool, void* out, float* lse) {
  const isd_config& c = ctx->cfg;
  AttnParams P;
  P.B = c.batch; P.Q = ctx->Q; P.N = c.stride; P.Hq = c.n_q_heads; P.Hkv = c.n_kv_heads; P.G = ctx->G;
  P.max_pages = c.max_pages_per_slot; P.num_pages = c.num_pages; P.sm_scale = ctx->sm_scale;
  P.ctx_len = st->ctx_len; P.n_ver = st->n_ver; P.active = st->active; P.page_table = st->page_table;
  P.slot_status = st->slot_status; P.global_status = ctx->global_status;
  P.q = (const __nv_bfloat16*)q; P.k_new = (const __nv_bfloat16*)k_new; P.v_new = (const __nv_bfloat16*)v_new;
  P.k_pool = (__nv_bfloat16*)k_pool; P.v_pool = (__nv_bfloat16*)v_pool; P.out = (__nv_bfloat16*)out; P.lse = lse;
  return P;
}

}  // namespace

int isd_launch_kv_append(isd_ctx* ctx, const isd_batch_state* st, const void* k_new, const void* v_new,
                         void* k_pool, void* v_pool, cudaStream_t stream) {
  const AttnParams P = make_params(ctx, st, nullptr, k_new, v_new, k_pool, v_pool, nullptr, nullptr);
  const cudaError_t e = isd_launch_pdl(kv_append_kernel, dim3(ctx->cfg.batch, ctx->cfg.n_kv_heads), dim3(128), 0, stream, P);
  ctx->launches++;
  return e == cudaSuccess ? ISD_OK : ISD_ERR_CUDA;
}

