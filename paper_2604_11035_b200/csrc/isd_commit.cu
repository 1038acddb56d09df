// isd_commit: KV commit / rollback and next-step state on the device (Algorithm 1 "commit KV
// cache"; Sec. 3.3 (2) trim-and-commit inside the stationary-batch loop; appendix renewal process).
//
// The rows a slot keeps (anchor + accepted proposals) are a logical prefix of its block, so dropping
// the rejected and [MASK] rows is a truncation: ctx_len += accept_len + 1.  Pages a slot lacks for
// its next block are popped from the top of the free stack in slot order; the order is fixed by an
// exclusive prefix sum of the requests, so the result does not depend on thread scheduling.  One CTA,
// no host round trip.
#include "isd_internal.cuh"

namespace {

constexpr int kCommitThreads = 1024;

struct CommitParams {
  int B, N, Q, max_pages, mask_token;
  int32_t* ctx_len;
  int32_t* n_ver;
  int32_t* block_tok;
  int32_t* q_row0;
  float* q_stats;
  int32_t* page_table;
  const int32_t* free_stack;
  int32_t* free_top;
  const uint8_t* active;
  uint32_t* slot_status;
  uint32_t* global_status;
  const int32_t* accept_len;
  const int32_t* repl_tok;
  const int32_t* new_prop_tok;
  const float* new_q_stats;
  uint32_t* step_counter;  // advanced by one after the commit when set
};

// exclusive prefix sum over the block; returns the block total through `total`
__device__ int block_exclusive_scan(int v, int* sm_warp, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int o = __shfl_up_sync(0xffffffffu, inc, off);
    if (lane >= off) inc += o;
  }
  if (lane == 31) sm_warp[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    int w = sm_warp[lane];
    int winc = w;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int o = __shfl_up_sync(0xffffffffu, winc, off);
      if (lane >= off) winc += o;
    }
    sm_warp[lane] = winc - w;  // exclusive warp offsets
    if (lane == 31) sm_warp[32] = winc;
  }
  __syncthreads();
  const int res = sm_warp[warp] + inc - v;
  total = sm_warp[32];
  __syncthreads();
  return res;
}

__global__ void __launch_bounds__(kCommitThreads) commit_kernel(const CommitParams P) {
  __shared__ int sm_warp[33];
  __shared__ int sm_popped;
  if (threadIdx.x == 0) sm_popped = 0;
  __syncthreads();
  const int top0 = *P.free_top;
  const int NP = P.N - 1;
  int carry = 0;  // pages requested by slots of earlier tiles (identical in every thread)
  for (int base = 0; base < P.B; base += kCommitThreads) {
    const int b = base + threadIdx.x;
    bool eligible = false;
    int need = 0, have = 0, a = 0, nv = 0, ctx_new = 0;
    if (b < P.B && P.active[b] && (P.slot_status[b] & ~ISD_ST_EMPTY_RESIDUAL) == 0) {
      a = P.accept_len[b];
      nv = P.n_ver[b];
      const int ctx = P.ctx_len[b];
      ctx_new = ctx + a + 1;
      have = (ctx + P.Q + ISD_PAGE - 1) / ISD_PAGE;
      const int want = (ctx_new + P.Q + ISD_PAGE - 1) / ISD_PAGE;
      if (want > P.max_pages) {
        atomicOr(&P.slot_status[b], ISD_ST_SLOT_CAPACITY);
        atomicOr(P.global_status, ISD_ST_SLOT_CAPACITY);
      } else {
        eligible = true;
        need = want - have;
      }
    }
    int total;
    const int before = carry + block_exclusive_scan(need, sm_warp, total);
    carry += total;
    if (eligible) {
      bool ok = true;
      if (need > 0) {
        if (before + need > top0) {
          ok = false;  // served requests are a prefix: every later request fails as well
          atomicOr(&P.slot_status[b], ISD_ST_POOL_EXHAUSTED);
          atomicOr(P.global_status, ISD_ST_POOL_EXHAUSTED);
        } else {
          for (int i = 0; i < need; ++i)
            P.page_table[(size_t)b * P.max_pages + have + i] = P.free_stack[top0 - 1 - (before + i)];
          atomicAdd(&sm_popped, need);
        }
      }
      if (ok) {
        const bool all_accepted = (a == nv);
        P.ctx_len[b] = ctx_new;
        P.n_ver[b] = all_accepted ? NP : 0;
        P.q_row0[b] = nv + 1;
        int32_t* bt = P.block_tok + (size_t)b * P.Q;
        bt[0] = P.repl_tok[b];
        for (int m = 1; m <= NP; ++m) {
          bt[m] = all_accepted ? P.new_prop_tok[(size_t)b * NP + m - 1] : P.mask_token;
          P.q_stats[((size_t)b * NP + m - 1) * 2 + 0] = P.new_q_stats[((size_t)b * NP + m - 1) * 2 + 0];
          P.q_stats[((size_t)b * NP + m - 1) * 2 + 1] = P.new_q_stats[((size_t)b * NP + m - 1) * 2 + 1];
        }
        for (int m = P.N; m < P.Q; ++m) bt[m] = P.mask_token;
      }
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    *P.free_top = top0 - sm_popped;
    if (P.step_counter) *P.step_counter += 1u;  // the next replay of a captured step draws fresh noise
  }
}

__global__ void release_kernel(int B, int Q, int max_pages, int32_t* ctx_len, int32_t* n_ver,
                               int32_t* page_table, int32_t* free_stack, int32_t* free_top,
                               uint8_t* active, const int32_t* slots, int n) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  int top = *free_top;
  for (int s = 0; s < n; ++s) {
    const int b = slots[s];
    if (b < 0 || b >= B || !active[b]) continue;
    const int have = (ctx_len[b] + Q + ISD_PAGE - 1) / ISD_PAGE;
    for (int i = 0; i < have; ++i) {
      free_stack[top++] = page_table[(size_t)b * max_pages + i];
      page_table[(size_t)b * max_pages + i] = -1;
    }
    active[b] = 0;
    ctx_len[b] = 0;
    n_ver[b] = 0;
  }
  *free_top = top;
}

}  // namespace

int isd_launch_commit(isd_ctx* ctx, isd_batch_state* st, const isd_verify_out* out, cudaStream_t stream) {
  const isd_config& c = ctx->cfg;
  CommitParams P;
  P.B = c.batch; P.N = c.stride; P.Q = ctx->Q; P.max_pages = c.max_pages_per_slot; P.mask_token = c.mask_token_id;
  P.ctx_len = st->ctx_len; P.n_ver = st->n_ver; P.block_tok = st->block_tok; P.q_row0 = st->q_row0;
  P.q_stats = st->q_stats; P.page_table = st->page_table; P.free_stack = st->free_stack; P.free_top = st->free_top;
  P.active = st->active; P.slot_status = st->slot_status; P.global_status = ctx->global_status;
  P.accept_len = out->accept_len; P.repl_tok = out->repl_tok; P.new_prop_tok = out->new_prop_tok;
  P.new_q_stats = out->new_q_stats;
  P.step_counter = ctx->step_counter;
  commit_kernel<<<1, kCommitThreads, 0, stream>>>(P);
  ctx->launches++;
  return cudaGetLastError() == cudaSuccess ? ISD_OK : ISD_ERR_CUDA;
}

int isd_launch_release(isd_ctx* ctx, isd_batch_state* st, const int32_t* slots, int32_t n, cudaStream_t stream) {
  const isd_config& c = ctx->cfg;
  release_kernel<<<1, 32, 0, stream>>>(c.batch, ctx->Q, c.max_pages_per_slot, st->ctx_len, st->n_ver,
                                       st->page_table, st->free_stack, st->free_top, st->active, slots, n);
  ctx->launches++;
  return cudaGetLastError() == cudaSuccess ? ISD_OK : ISD_ERR_CUDA;
}
