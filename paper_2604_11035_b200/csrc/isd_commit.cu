// isd_commit as a kernel of its own (the stand-alone entry point, and steps whose verification does not
// commit by itself) and isd_release.  The commit itself is in isd_commit.cuh.
#include "isd_commit.cuh"

namespace {

constexpr int kCommitThreads = 1024;

__global__ void __launch_bounds__(kCommitThreads) commit_kernel(const CommitParams P) {
  __shared__ int sm_warp[33];
  __shared__ int sm_popped;
  pdl_wait();
  commit_block(P, sm_warp, &sm_popped);
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
  const CommitParams P = make_commit_params(ctx, st, out);
  const cudaError_t e = isd_launch_pdl(commit_kernel, dim3(1), dim3(kCommitThreads), 0, stream, P);
  ctx->launches++;
  return e == cudaSuccess ? ISD_OK : ISD_ERR_CUDA;
}

int isd_launch_release(isd_ctx* ctx, isd_batch_state* st, const int32_t* slots, int32_t n, cudaStream_t stream) {
  const isd_config& c = ctx->cfg;
  release_kernel<<<1, 32, 0, stream>>>(c.batch, ctx->Q, c.max_pages_per_slot, st->ctx_len, st->n_ver,
                                       st->page_table, st->free_stack, st->free_top, st->active, slots, n);
  ctx->launches++;
  return cudaGetLastError() == cudaSuccess ? ISD_OK : ISD_ERR_CUDA;
}
