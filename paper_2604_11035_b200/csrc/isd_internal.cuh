// Internal declarations shared by the ISD kernels (sm_100a).  Not part of the C ABI.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/isd.h"

#define ISD_PAGE 16
#define ISD_HEAD_DIM 128
#define ISD_MAX_Q 31
#define ISD_NUM_SMS_DEFAULT 148

// Philox stream tags (counter word 3 = tag << 16 | position)
#define ISD_TAG_ACCEPT 0u
#define ISD_TAG_FINAL 1u
#define ISD_TAG_PROPOSE 2u

// internal status bit (not part of the public set): a bounded wait inside a kernel ran out
#ifndef ISD_ST_KERNEL_TIMEOUT
#define ISD_ST_KERNEL_TIMEOUT 0x80000000u
#endif

// score gap below which two Gumbel-max candidates are re-judged in fp64
#define ISD_TIE_EPS 1e-3f

// Partial result of one (slot, row, split) CTA of the row-statistics pass.
struct RowPartial {
  float m;        // max of the scaled logits in the chunk
  float s;        // sum of exp(l - m) over the chunk
  float raw_max;  // max of the raw logits in the chunk ...
  int idx;        // ... and the lowest index that attains it (-1: none)
};

// Partial result of one (slot, sampled row, split) CTA of the sampling pass: the two best noisy scores.
struct SamplePartial {
  float best1;
  int idx1;
  float best2;
  int idx2;
};

struct isd_ctx {
  isd_config cfg;
  int device;
  int num_sms;
  int Q;            // 2N - 1
  int G;            // Hq / Hkv
  float sm_scale;
  // ---- verify scratch
  int row_splits;        // CTAs per logits row in the row pass
  int sample_splits;     // CTAs per sampled row in the sampling pass
  RowPartial* row_part;  // [B, Q, row_splits]
  SamplePartial* samp_part;  // [B, N, sample_splits]
  int* row_ticket;       // [B] arrivals of the row pass
  int* samp_ticket;      // [B, N] arrivals of the sampling pass
  int* reject_pos;       // [B] -1 = slot frozen (nothing to sample), 0 = nothing rejected, j = first rejected proposal
  int* row_arg;          // [B, Q] argmax of every valid row (seeds the sampling pass)
  float* lse_p_rej;      // [B] LSE of the anchor row that rejected
  // ---- attention scratch
  int attn_ctas;         // persistent CTAs of the tensor-core kernel
  float* attn_part_o;    // [attn_ctas * 2, 128, 128] un-normalised partial outputs
  float* attn_part_ml;   // [attn_ctas * 2, 128, 2]   running max / sum of each partial row
  void* tmap_k;          // host-side state of the tensor-core attention (tensor maps of the pools seen so far)
  // ---- optional instrumentation events (owned by the caller)
  cudaEvent_t ev_attn0, ev_attn1, ev_verify0, ev_verify1;
  // ---- scratch of the top-k / top-p filtered verification (cfg.top_k > 0)
  float* topk_val;       // [B, Q, ISD_MAX_TOP_K]
  int* topk_idx;         // [B, Q, ISD_MAX_TOP_K]
  int* topk_n;           // [B, Q]   (each of the three twice: this call's lists and the previous call's)
  int topk_cur;          // which half the next call writes
  const void* topk_prev_rows;  // logits_cur of the previous filtered call (whose lists the other half holds)
  uint32_t topk_prev_step;     // and its step number
  unsigned long long* topk_q_key;  // [B, pieces, ISD_MAX_TOP_K] piece lists of a proposal-law row (as sort keys)
  int* topk_q_n;         // [B, pieces], then the slot decisions, supports and row tickets of the accept phase
  double* topk_nuc_lse;  // [B, Q] log-normaliser of every row's filtered law
  // ---- isd_lora_linear: readiness flags of the row blocks of t, then one counter (all zero between launches)
  uint32_t* lora_flags;
  // ---- optional device-resident step counter (CUDA-graph replay), owned by the caller
  uint32_t* step_counter;
  // ---- status
  uint32_t* global_status;  // [1]
  int64_t launches;
};

// -------------------------------------------------------------------------------------------------
// Device helpers
// -------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    if (r > 0) {
      k0 += 0x9E3779B9u;
      k1 += 0xBB67AE85u;
    }
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0;
    const uint32_t n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
  }
  return make_uint4(c0, c1, c2, c3);
}

__device__ __forceinline__ uint32_t philox_word(const uint4& v, int w) {
  return w == 0 ? v.x : (w == 1 ? v.y : (w == 2 ? v.z : v.w));
}

// Standard Gumbel variate from a 32-bit word: u' = ((w >> 8) + 0.5) 2^-24, g = -ln(-ln u').
// Evaluated through 1 - u' when u' > 1/2 so that both branches are exact on the lattice.
__device__ __forceinline__ float gumbel_f32(uint32_t w) {
  const uint32_t k = w >> 8;
  float t;
  if (k >= (1u << 23)) {
    const float v = ((float)(0xFFFFFFu - k) + 0.5f) * 0x1p-24f;  // 1 - u', exact
    t = -log1pf(-v);
  } else {
    const float u = ((float)k + 0.5f) * 0x1p-24f;  // exact
    t = -logf(u);
  }
  return -logf(t);
}

__device__ __forceinline__ double gumbel_f64(uint32_t w) {
  const double u = ((double)(w >> 8) + 0.5) * 0x1p-24;
  return -log(-log(u));
}

__device__ __forceinline__ float bf16_bits_to_f32(uint32_t h16) { return __uint_as_float(h16 << 16); }

__device__ __forceinline__ float load_logit(const void* base, int dtype, size_t idx) {
  if (dtype == ISD_LOGITS_F32) return reinterpret_cast<const float*>(base)[idx];
  return bf16_bits_to_f32(reinterpret_cast<const uint16_t*>(base)[idx]);
}

__device__ __forceinline__ uint4 ld_stream_16B(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// Packed fp32x2 arithmetic (two lanes per instruction on sm_100) and 3-input max
__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// -------------------------------------------------------------------------------------------------
// mbarrier / bulk-copy helpers for shared-memory rings (one producer thread, many consumers)
// -------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t ring_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void ring_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void ring_mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void ring_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait on a phase parity; false when the limit expires (the caller raises a status bit and leaves).
__device__ __forceinline__ bool ring_mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < (1u << 24); ++i) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    if (ok) return true;
  }
  return false;
}
// The same wait where the phase has normally completed already: one probe, then the bounded loop.
__device__ __forceinline__ bool mbar_wait_likely(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  if (__builtin_expect(ok != 0, 1)) return true;
  return ring_mbar_wait(bar, parity);
}
// Contiguous global -> shared copy (16-byte aligned addresses, size a multiple of 16) that signals `bar`.
__device__ __forceinline__ void ring_bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Ordering of (score, index) candidates: higher score wins, ties go to the lower index.
__device__ __forceinline__ bool cand_better(float sa, int ia, float sb, int ib) {
  if (ib < 0) return ia >= 0;
  if (ia < 0) return false;
  return sa > sb || (sa == sb && ia < ib);
}

struct Top2 {
  float s1;
  int i1;
  float s2;
  int i2;
  __device__ __forceinline__ void init() {
    s1 = -INFINITY; i1 = -1; s2 = -INFINITY; i2 = -1;
  }
  __device__ __forceinline__ void push(float s, int i) {
    if (cand_better(s, i, s1, i1)) {
      s2 = s1; i2 = i1; s1 = s; i1 = i;
    } else if (cand_better(s, i, s2, i2)) {
      s2 = s; i2 = i;
    }
  }
  __device__ __forceinline__ void merge(float os1, int oi1, float os2, int oi2) {
    push(os1, oi1);
    push(os2, oi2);
  }
};

__device__ __forceinline__ void warp_merge_top2(Top2& t) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float os1 = __shfl_xor_sync(0xffffffffu, t.s1, off);
    const int oi1 = __shfl_xor_sync(0xffffffffu, t.i1, off);
    const float os2 = __shfl_xor_sync(0xffffffffu, t.s2, off);
    const int oi2 = __shfl_xor_sync(0xffffffffu, t.i2, off);
    t.merge(os1, oi1, os2, oi2);
  }
}

// (m, s) pairs of an online softmax: combine two partial sums of exp(l - m).
__device__ __forceinline__ void lse_merge(float& m, float& s, float om, float os) {
  const float nm = fmaxf(m, om);
  if (nm == -INFINITY) {
    s = 0.f;
    m = nm;
    return;
  }
  s = s * __expf(m - nm) + os * __expf(om - nm);
  m = nm;
}

// -------------------------------------------------------------------------------------------------
// Host-side launchers implemented in the .cu files
// -------------------------------------------------------------------------------------------------
int isd_launch_verify(isd_ctx* ctx, const isd_batch_state* st, const void* logits_cur,
                      const void* q_prev_logits, uint32_t step, const isd_verify_out* out,
                      cudaStream_t stream);
int isd_verify_topk_create(isd_ctx* ctx);
void isd_verify_topk_destroy(isd_ctx* ctx);
int isd_launch_verify_topk(isd_ctx* ctx, const isd_batch_state* st, const void* logits_cur,
                           const void* q_prev_logits, uint32_t step, const isd_verify_out* out,
                           cudaStream_t stream);
int isd_launch_lora_linear(isd_ctx* ctx, const isd_lora_args* a, cudaStream_t stream);
int isd_lora_create(isd_ctx* ctx);
void isd_lora_destroy(isd_ctx* ctx);
int isd_launch_commit(isd_ctx* ctx, isd_batch_state* st, const isd_verify_out* out, cudaStream_t stream);
int isd_launch_release(isd_ctx* ctx, isd_batch_state* st, const int32_t* slots, int32_t n,
                       cudaStream_t stream);
int isd_launch_attn_plain(isd_ctx* ctx, const isd_batch_state* st, const void* q, const void* k_new,
                          const void* v_new, void* k_pool, void* v_pool, void* out, float* lse,
                          cudaStream_t stream);
int isd_launch_attn_tc(isd_ctx* ctx, const isd_batch_state* st, const void* q, const void* k_new,
                       const void* v_new, void* k_pool, void* v_pool, void* out, float* lse,
                       cudaStream_t stream);
int isd_attn_tc_scratch_bytes(const isd_ctx* ctx, size_t* part_o, size_t* part_ml);
