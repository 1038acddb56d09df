// Device side of isd_commit, shared by the stand-alone commit kernel and by the last CTA of the verification
// kernels inside isd_step (Algorithm 1 "commit KV cache"; Sec. 3.3 (2) trim-and-commit inside the
// stationary-batch loop; appendix renewal process).
//
// The rows a slot keeps (anchor + accepted proposals) are a logical prefix of its block, so dropping
// the rejected and [MASK] rows is a truncation: ctx_len += accept_len + 1.  Pages a slot lacks for
// its next block are popped from the top of the free stack in slot order; the order is fixed by an
// exclusive prefix sum of the requests, so the result does not depend on thread scheduling.  One CTA,
// no host round trip.
#pragma once
#include "isd_internal.cuh"

namespace {

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

inline CommitParams make_commit_params(const isd_ctx* ctx, const isd_batch_state* st, const isd_verify_out* out) {
  const isd_config& c = ctx->cfg;
  CommitParams P;
  P.B = c.batch; P.N = c.stride; P.Q = ctx->Q; P.max_pages = c.max_pages_per_slot; P.mask_token = c.mask_token_id;
  P.ctx_len = st->ctx_len; P.n_ver = st->n_ver; P.block_tok = st->block_tok; P.q_row0 = st->q_row0;
  P.q_stats = st->q_stats; P.page_table = st->page_table; P.free_stack = st->free_stack; P.free_top = st->free_top;
  P.active = st->active; P.slot_status = st->slot_status; P.global_status = ctx->global_status;
  P.accept_len = out->accept_len; P.repl_tok = out->repl_tok; P.new_prop_tok = out->new_prop_tok;
  P.new_q_stats = out->new_q_stats;
  P.step_counter = ctx->step_counter;
  return P;
}

// exclusive prefix sum over the block (blockDim.x a multiple of 32, at most 1024); the block total comes back
// through `total`.  sm_warp: 33 ints of shared memory.
__device__ __forceinline__ int block_exclusive_scan(int v, int* sm_warp, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = (int)blockDim.x >> 5;
  int inc = v;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int o = __shfl_up_sync(0xffffffffu, inc, off);
    if (lane >= off) inc += o;
  }
  if (lane == 31) sm_warp[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    int w = lane < n_warps ? sm_warp[lane] : 0;
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

// The commit of the whole batch by ONE CTA (every thread of it must call; blockDim.x a multiple of 32).
// What the verification kernels produced is read from L2 (ld.cg): inside isd_step the caller is a CTA of the
// very kernel whose other CTAs wrote it.
// sm_warp: 33 ints, sm_popped: 1 int of shared memory.
__device__ __forceinline__ void commit_block(const CommitParams& P, int* sm_warp, int* sm_popped) {
  if (threadIdx.x == 0) *sm_popped = 0;
  __syncthreads();
  const int top0 = *P.free_top;
  const int NP = P.N - 1;
  int carry = 0;  // pages requested by slots of earlier tiles (identical in every thread)
  for (int base = 0; base < P.B; base += (int)blockDim.x) {
    const int b = base + threadIdx.x;
    bool eligible = false;
    int need = 0, have = 0, a = 0, nv = 0, ctx_new = 0;
    if (b < P.B && P.active[b] && (__ldcg(P.slot_status + b) & ~ISD_ST_EMPTY_RESIDUAL) == 0) {
      a = __ldcg(P.accept_len + b);
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
          atomicAdd(sm_popped, need);
        }
      }
      if (ok) {
        const bool all_accepted = (a == nv);
        P.ctx_len[b] = ctx_new;
        P.n_ver[b] = all_accepted ? NP : 0;
        P.q_row0[b] = nv + 1;
        int32_t* bt = P.block_tok + (size_t)b * P.Q;
        bt[0] = __ldcg(P.repl_tok + b);
        for (int m = 1; m <= NP; ++m) {
          bt[m] = all_accepted ? __ldcg(P.new_prop_tok + (size_t)b * NP + m - 1) : P.mask_token;
          if (!all_accepted) continue;  // no proposals were made after a rejection: nothing to keep statistics of
          P.q_stats[((size_t)b * NP + m - 1) * 2 + 0] = __ldcg(P.new_q_stats + ((size_t)b * NP + m - 1) * 2 + 0);
          P.q_stats[((size_t)b * NP + m - 1) * 2 + 1] = __ldcg(P.new_q_stats + ((size_t)b * NP + m - 1) * 2 + 1);
        }
        for (int m = P.N; m < P.Q; ++m) bt[m] = P.mask_token;
      }
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    *P.free_top = top0 - *sm_popped;
    if (P.step_counter) *P.step_counter += 1u;  // the next replay of a captured step draws fresh noise
  }
}

}  // namespace
