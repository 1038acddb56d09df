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

// default time limit of a device-side wait (isd_set_wait_limit changes it per context)
#define ISD_DEFAULT_WAIT_NS 250000000ull

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
  RowPartial* row_part;  // [B, Q, row_splits, worker warps of a CTA]
  SamplePartial* samp_part;  // [B, N, sample_splits]
  int* samp_ticket;      // [B, N] arrivals of the sampling pass
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
  // ---- isd_step: arrivals of the last verification kernel's CTAs (the last one commits), zero between calls
  int* step_ticket;
  // ---- time limit of every device-side wait, nanoseconds
  unsigned long long wait_ns;
  // ---- status
  uint32_t* global_status;  // [1]
  int64_t launches;
};

// -------------------------------------------------------------------------------------------------
// Device helpers
// -------------------------------------------------------------------------------------------------
// 32 x 32 -> 64 bit product as one instruction (both halves are needed by every Philox round)
__device__ __forceinline__ void mul_wide_u32(uint32_t a, uint32_t b, uint32_t& hi, uint32_t& lo) {
  uint64_t p;
  asm("mul.wide.u32 %0, %1, %2;" : "=l"(p) : "r"(a), "r"(b));
  asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(p));
}

__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    if (r > 0) {
      k0 += 0x9E3779B9u;
      k1 += 0xBB67AE85u;
    }
    uint32_t hi0, lo0, hi1, lo1;
    mul_wide_u32(0xD2511F53u, c0, hi0, lo0);
    mul_wide_u32(0xCD9E8D57u, c2, hi1, lo1);
    const uint32_t n0 = hi1 ^ c1 ^ k0;
    const uint32_t n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
  }
  return make_uint4(c0, c1, c2, c3);
}

// The ten round keys of a Philox key (k0 + r * 0x9E3779B9, k1 + r * 0xBB67AE85), computed once on the host and
// passed as kernel parameters: inside the sampling loops a round is then two wide multiplies and two three-input
// XORs whose third operand comes straight from the constant bank.
struct PhiloxKeys {
  uint32_t k[20];
};
inline void philox_round_keys(uint64_t seed, PhiloxKeys& rk) {
  uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
  for (int r = 0; r < 10; ++r) {
    rk.k[2 * r] = k0;
    rk.k[2 * r + 1] = k1;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
}
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, const PhiloxKeys& rk) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    uint32_t hi0, lo0, hi1, lo1;
    mul_wide_u32(0xD2511F53u, c0, hi0, lo0);
    mul_wide_u32(0xCD9E8D57u, c2, hi1, lo1);
    const uint32_t n0 = hi1 ^ c1 ^ rk.k[2 * r];
    const uint32_t n2 = hi0 ^ c3 ^ rk.k[2 * r + 1];
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
// Bounded waits.  Every device-side wait of the library (an mbarrier phase, a readiness counter written by
// another CTA) polls through this routine: after the first 64 failed probes it reads the nanosecond clock
// every 64 probes and gives up once `budget_ns` has passed since then.  The caller then raises
// ISD_ST_KERNEL_TIMEOUT, stops issuing work, waits (bounded again) for its copies in flight, frees what it
// holds and returns, so the context stays usable.  `abort_flag` (may be null) is the CTA's shared flag: a wait
// also ends when another thread of the CTA has given up, and raises it when its own limit runs out.
// -------------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned long long isd_now_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
template <class Probe>
__device__ __forceinline__ bool isd_bounded_wait(unsigned long long budget_ns, volatile int* abort_flag, Probe probe) {
  unsigned long long t0 = 0;
  for (uint32_t i = 1;; ++i) {
    if (probe()) return true;
    if ((i & 63u) == 0u) {
      if (abort_flag && *abort_flag) return false;
      const unsigned long long now = isd_now_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > budget_ns) {
        if (abort_flag) *abort_flag = 1;
        return false;
      }
    }
  }
}

// Programmatic dependent launch: the kernels of a step are launched with the programmatic-serialisation
// attribute, so a kernel's CTAs may become resident while the kernel before it in the stream is still draining.
// pdl_wait() returns once that kernel has completed and its writes are visible; every kernel executes it before
// it reads anything an earlier kernel wrote and before any return, so completion stays transitive along the chain.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

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
__device__ __forceinline__ bool ring_mbar_probe(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait on a phase parity; false when the time limit expires (the caller raises a status bit and leaves).
__device__ __forceinline__ bool ring_mbar_wait(uint32_t bar, uint32_t parity, unsigned long long budget_ns) {
  return isd_bounded_wait(budget_ns, nullptr, [&]() { return ring_mbar_probe(bar, parity); });
}
// The same wait where the phase has normally completed already: one probe, then the bounded loop.
__device__ __forceinline__ bool mbar_wait_likely(uint32_t bar, uint32_t parity, unsigned long long budget_ns) {
  if (__builtin_expect(ring_mbar_probe(bar, parity), 1)) return true;
  return ring_mbar_wait(bar, parity, budget_ns);
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
};

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
// Host side: launch with the programmatic-serialisation attribute (see pdl_wait above)
// -------------------------------------------------------------------------------------------------
template <typename... KArgs, typename... Args>
inline cudaError_t isd_launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                  Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// -------------------------------------------------------------------------------------------------
// Host-side launchers implemented in the .cu files
// -------------------------------------------------------------------------------------------------
// commit_st != nullptr: the last CTA of the last verification kernel also commits (isd_step)
int isd_launch_verify(isd_ctx* ctx, const isd_batch_state* st, const void* logits_cur,
                      const void* q_prev_logits, uint32_t step, const isd_verify_out* out,
                      cudaStream_t stream, isd_batch_state* commit_st = nullptr);
int isd_verify_topk_create(isd_ctx* ctx);
void isd_verify_topk_destroy(isd_ctx* ctx);
// commit_st != nullptr: the row kernel's last CTA commits when no decide kernel follows it; *committed says whether
int isd_launch_verify_topk(isd_ctx* ctx, const isd_batch_state* st, const void* logits_cur,
                           const void* q_prev_logits, uint32_t step, const isd_verify_out* out,
                           cudaStream_t stream, isd_batch_state* commit_st = nullptr, bool* committed = nullptr);
int isd_launch_lora_linear(isd_ctx* ctx, const isd_lora_args* a, cudaStream_t stream);
int isd_lora_create(isd_ctx* ctx);
void isd_lora_destroy(isd_ctx* ctx);
int isd_launch_commit(isd_ctx* ctx, isd_batch_state* st, const isd_verify_out* out, cudaStream_t stream);
int isd_launch_release(isd_ctx* ctx, isd_batch_state* st, const int32_t* slots, int32_t n,
                       cudaStream_t stream);
int isd_launch_kv_append(isd_ctx* ctx, const isd_batch_state* st, const void* k_new, const void* v_new,
                         void* k_pool, void* v_pool, cudaStream_t stream);
int isd_launch_attn_tc(isd_ctx* ctx, const isd_batch_state* st, const void* q, const void* k_new,
                       const void* v_new, void* k_pool, void* v_pool, void* out, float* lse,
                       cudaStream_t stream);
int isd_attn_tc_scratch_bytes(const isd_ctx* ctx, size_t* part_o, size_t* part_ml);
