// isd_verify: vocab-wide softmax statistics, p/q introspective acceptance, residual resample /
// bonus token and next proposals (Algorithm 1; Sec. 3.2; Sec. 3.3 (3) fused verification with
// online softmax and Gumbel-max correction).
//
// Two launches, neither of which waits on anything:
//   1. verify_rows_kernel   one CTA per (slot, block row, split): a single streaming pass over the
//      logits row that yields the online-softmax pair (max, sum) -> LSE and the argmax of the row.
//      Every row has the same role here, so the kernel is a lean HBM stream; every warp ends with one
//      store of its partial and nothing else (no merge, no fence, no ticket).
//   2. verify_sample_kernel one CTA per (slot, sampled row, split).  At its head one warp merges the
//      partials of the slot's rows, runs the accept tests of all proposals at once (Algorithm 1's
//      sequence ends at the first that fails) and, in the CTA with split 0, writes every output that
//      needs no random sample: accept flags, alpha, accept length, the accepted tokens, argmax
//      proposals and the proposal-law statistics.  Then each slot draws exactly one token for its
//      emission: the replacement from normalize(max(0, p - q)) when a proposal was rejected, else the
//      bonus / free token from the row of the last clean token; with sampled proposals the N - 1 MASK
//      rows are drawn here too.  The pass reads the row again.
//
// Gumbel noise is a pure function of (seed, step, slot, tag, position, vocab index), so any
// reduction order gives the same sample, and it is evaluated only for elements that can still win.
// The sampling pass starts from the true noisy score of the row's argmax (its logit is the row's maximum), which
// is a lower bound of the winner's score from the first element on.  (1) No variate on the 24-bit
// lattice exceeds 25 ln 2 = 17.33, so a group of four logits whose maximum is more than 17.34 below
// the running best needs no random numbers at all; the groups that survive are compacted into a
// per-warp queue so that the Philox work runs on full warps.  (2) With E = -ln u' >= 1 - u', a
// queued element whose cheap bound cannot reach the running best is skipped before any logarithm.
// The two best candidates of a row are re-judged in fp64 when their fp32 scores are closer than
// ISD_TIE_EPS.
#include "isd_internal.cuh"
#include "isd_stream.cuh"
#include "isd_commit.cuh"

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kGumbelMax = 17.34f;  // > 25 ln 2, the largest variate of the 24-bit lattice

struct VerifyParams {
  int B, N, Q, V;
  int logits_dtype, q_mode, propose_mode;
  float inv_t, tau;
  unsigned long long wait_ns;  // time limit of a device-side wait
  PhiloxKeys rk;               // round keys of the seed
  uint32_t seed_lo, seed_hi, step;
  const uint32_t* step_dev;  // when set, the step number is read from here (CUDA-graph replay) instead of `step`
  int row_splits, sample_splits;
  const int32_t* n_ver;
  const uint8_t* active;
  const int32_t* block_tok;
  const int32_t* q_row0;
  const float* q_stats;
  uint32_t* slot_status;
  uint32_t* global_status;
  const void* logits_cur;
  const void* q_prev;
  isd_verify_out out;
  RowPartial* row_part;
  SamplePartial* samp_part;
  int* samp_ticket;
  // isd_step: the CTA of the sampling pass that finishes last commits the batch (fuse_commit != 0)
  int fuse_commit;
  int rows_early;  // isd_step: the row pass starts before the kernel ahead of it has completed (see verify_rows_kernel)
  int* step_ticket;
  CommitParams commit;
};

// rows nv .. nv + rows_sampled - 1 of a slot are drawn by the sampling pass
__device__ __forceinline__ int rows_sampled(const VerifyParams& P) { return P.propose_mode == 0 ? P.N : 1; }
__device__ __forceinline__ uint32_t step_of(const VerifyParams& P) { return P.step_dev ? *P.step_dev : P.step; }

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Order-preserving map float -> unsigned (larger float = larger code; code 0 is below every float and
// decodes to a NaN, which fmaxf ignores): lets the running best score live behind atomicMax.
__device__ __forceinline__ unsigned enc_ordered(float f) {
  const unsigned b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float dec_ordered(unsigned u) {
  return __uint_as_float((u & 0x80000000u) ? (u ^ 0x80000000u) : ~u);
}

// A row piece streamed through shared memory with per-thread asynchronous copies.  Every thread
// fetches its own logits of the next kDepth iterations ahead of time (no registers held) and later
// reads back exactly what it fetched itself, so no barrier is needed.  The load latency, which bounds
// a pass that issues one load per iteration and then computes on it, disappears behind the iterations
// in between.  U = groups of eight logits per thread and iteration (group g of thread t covers elements
// base + g * kThreads * 8 + t * 8): the bookkeeping of an iteration is paid once for all of them.
template <int DT, int U, int RING_BYTES>
struct RowStream {
  static constexpr int kElt = DT == ISD_LOGITS_BF16 ? 2 : 4;
  static constexpr int kVec = kElt / 2;                        // 16-byte vectors per group of eight logits
  static constexpr int kGroupBytes = kThreads * 8 * kElt;      // one group of every thread
  static constexpr int kStageBytes = U * kGroupBytes;
  static constexpr int kDepth = RING_BYTES / kStageBytes;
  static constexpr int kGroupStep = kThreads * 8;              // elements between a thread's groups
  static constexpr int kStep = U * kGroupStep;                 // elements per iteration of the CTA
  static_assert(kDepth >= 2 && (kDepth & (kDepth - 1)) == 0, "ring depth must be a power of two");
  uint32_t sbase;   // shared-memory address of this thread's first vector in stage 0
  uint32_t soff;    // byte offset of the stage that is read (and refilled) next
  const char* src;  // global address of this thread's next fetch ...
  int e_fetch;      // ... and its element index
  int hi;

  __device__ __forceinline__ void fetch(uint32_t stage_off) {
#pragma unroll
    for (int g = 0; g < U; ++g) {
      if (e_fetch + g * kGroupStep < hi) {
#pragma unroll
        for (int v = 0; v < kVec; ++v)
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sbase + stage_off + g * kGroupBytes + 16 * v),
                       "l"(src + g * kGroupBytes + 16 * v)
                       : "memory");
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");  // one group per iteration, empty or not
    src += kStageBytes;
    e_fetch += kStep;
  }
  __device__ __forceinline__ void start(uint4* ring, const char* row, int lo, int hi_) {
    sbase = (uint32_t)__cvta_generic_to_shared(ring) + threadIdx.x * 16 * kVec;
    soff = 0;
    e_fetch = lo + threadIdx.x * 8;
    src = row + (size_t)e_fetch * kElt;
    hi = hi_;
#pragma unroll
    for (int s = 0; s < kDepth; ++s) fetch(s * kStageBytes);
  }
  // this thread's logits of the iteration that was fetched kDepth fetches ago (the caller knows which of
  // them exist); refills the stage
  __device__ __forceinline__ void next(float (&l)[U][8]) {
    asm volatile("cp.async.wait_group %0;" ::"n"(kDepth - 1) : "memory");
#pragma unroll
    for (int g = 0; g < U; ++g) {
      uint4 a, b = make_uint4(0u, 0u, 0u, 0u);
      const uint32_t addr = sbase + soff + g * kGroupBytes;
      asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w) : "r"(addr) : "memory");
      if (kVec == 2)
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w) : "r"(addr + 16) : "memory");
      unpack8<DT>(a, b, l[g]);
    }
    fetch(soff);
    soff = (soff + kStageBytes) & (RING_BYTES - 1);
  }
  __device__ __forceinline__ void finish() const { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
};
constexpr int kSampleRingBytes = 16384;  // sampling pass: one group per iteration

__device__ __forceinline__ void chunk_range(int V, int splits, int split, int& lo, int& hi) {
  // chunks are multiples of 8 * kThreads elements so that every thread's vector stays aligned
  const int per = ((V + splits - 1) / splits + 8 * kThreads - 1) / (8 * kThreads) * (8 * kThreads);
  lo = split * per;
  hi = min(V, lo + per);
}

// Top-2 merges ----------------------------------------------------------------------------------------
// The two best of the union of the lanes' candidate pairs, in every lane: the winner is the best first
// candidate (highest score, lowest index among equals), the runner-up the best of the other lanes' first
// candidates and the winner lane's second.  On order-preserving integer codes of the scores each place is one
// max- and one min-reduction of the warp, where five shuffle rounds of compare-and-swap on pairs cost some
// three hundred dependent instructions at the end of every CTA.  (Indices are distinct across lanes: they are
// different elements of a row.)
__device__ __forceinline__ void warp_top2(Top2& t) {
  const unsigned full = 0xffffffffu;
  const unsigned k1 = t.i1 >= 0 ? enc_ordered(t.s1) : 0u;
  const unsigned K1 = __reduce_max_sync(full, k1);
  const int I1 = __reduce_min_sync(full, (t.i1 >= 0 && k1 == K1) ? t.i1 : 0x7FFFFFFF);
  const bool won = t.i1 >= 0 && t.i1 == I1;
  const float cs = won ? t.s2 : t.s1;
  const int ci = won ? t.i2 : t.i1;
  const unsigned k2 = ci >= 0 ? enc_ordered(cs) : 0u;
  const unsigned K2 = __reduce_max_sync(full, k2);
  const int I2 = __reduce_min_sync(full, (ci >= 0 && k2 == K2) ? ci : 0x7FFFFFFF);
  t.s1 = K1 ? dec_ordered(K1) : -INFINITY; t.i1 = K1 ? I1 : -1;
  t.s2 = K2 ? dec_ordered(K2) : -INFINITY; t.i2 = K2 ? I2 : -1;
}

// Over the 8 worker warps of a CTA; the result is valid in warp 0.  One barrier: the arrays are not touched
// again before the next CTA-wide barrier of the caller.
__device__ __forceinline__ void block_merge_top2(Top2& t, float* sm_s1, int* sm_i1, float* sm_s2, int* sm_i2) {
  warp_top2(t);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) { sm_s1[warp] = t.s1; sm_i1[warp] = t.i1; sm_s2[warp] = t.s2; sm_i2[warp] = t.i2; }
  worker_sync();
  if (warp == 0) {
    t.init();
    if (lane < kThreads / 32) { t.s1 = sm_s1[lane]; t.i1 = sm_i1[lane]; t.s2 = sm_s2[lane]; t.i2 = sm_i2[lane]; }
    warp_top2(t);
  }
}

// fp64 score of vocabulary index i of a Gumbel row: logit * invT + g
__device__ double noisy_score_f64(const VerifyParams& P, const void* row, int i, uint32_t step, uint32_t slot, uint32_t tagpos) {
  const uint4 r = philox4x32_10((uint32_t)i >> 2, step, slot, tagpos, P.seed_lo, P.seed_hi);
  const double l = (double)load_logit(row, P.logits_dtype, (size_t)i) * (double)P.inv_t;
  return l + gumbel_f64(philox_word(r, i & 3));
}

// Online softmax of a thread's share of a row: S = sum exp((l - M) * invT) in the log2 domain, plain
// scalar FFMA / ex2 / FADD with four independent partial sums (the packed fp32x2 forms cost more in
// register-pair moves here than they save).  The reference point M is the running maximum of the WARP,
// not of the thread: the warp agrees on it with one integer max-reduction per iteration, which makes
// "the maximum grew" a warp-uniform and genuinely rare branch (about ln(iterations) times per row),
// where per-thread maxima would send some lane of the warp into it in most iterations.
struct OnlineSoftmax {
  float M, neg_ms, scale2;
  int Mkey;
  float S0, S1, S2, S3;
  __device__ __forceinline__ void init(float inv_t) {
    scale2 = inv_t * kLog2e;  // raw logit -> log2 domain
    M = -INFINITY;            // running max of the raw logits seen by the warp
    Mkey = ord_key(M);
    neg_ms = 0.f;             // -M * scale2 (0 while M = -inf, so that -inf logits give e = 0)
    S0 = S1 = S2 = S3 = 0.f;
  }
  __device__ __forceinline__ void raise_to(float new_m, int new_key) {
    const float f = (M == -INFINITY) ? 0.f : ex2f((M - new_m) * scale2);
    S0 *= f; S1 *= f; S2 *= f; S3 *= f;
    M = new_m;
    Mkey = new_key;
    neg_ms = -M * scale2;
  }
  __device__ __forceinline__ void add8(const float (&l)[8]) {
    S0 += ex2f(fmaf(l[0], scale2, neg_ms));
    S1 += ex2f(fmaf(l[1], scale2, neg_ms));
    S2 += ex2f(fmaf(l[2], scale2, neg_ms));
    S3 += ex2f(fmaf(l[3], scale2, neg_ms));
    S0 += ex2f(fmaf(l[4], scale2, neg_ms));
    S1 += ex2f(fmaf(l[5], scale2, neg_ms));
    S2 += ex2f(fmaf(l[6], scale2, neg_ms));
    S3 += ex2f(fmaf(l[7], scale2, neg_ms));
  }
  __device__ __forceinline__ float sum() const { return (S0 + S1) + (S2 + S3); }
};

// Worker side of one streaming pass over elements [lo, hi) of a logits row: online softmax (m_nat, S
// relative to the warp's maximum) and this thread's argmax candidate of the raw logits.  A thread
// records (value, position) only when one of its elements sets a new maximum of the warp, strictly
// above everything the warp saw before; merging the candidates by (value, lowest index) gives the first
// occurrence of the row maximum.  Thread t reads vectors t, t + kThreads, ... of a stage (bf16: two
// groups of eight logits per stage; fp32: one group from two adjacent vectors).
template <int DT>
__device__ __forceinline__ bool row_pass(const VerifyParams& P, RowRing& R, const char* row, int lo, int hi,
                                         float& warp_max, float& S_out, float& raw_max, int& raw_idx) {
  constexpr int kElt = DT == ISD_LOGITS_BF16 ? 2 : 4;
  constexpr int U = DT == ISD_LOGITS_BF16 ? 2 : 1;      // groups of eight logits per thread and stage
  constexpr int kStageElems = kRowStageBytes / kElt;
  constexpr int kGroupStep = kStageElems / U;           // elements between a thread's groups
  const uint32_t full0 = ring_smem_u32(R.full), empty0 = ring_smem_u32(R.empty);
  const uint32_t mine = ring_smem_u32(R.stage) + threadIdx.x * (DT == ISD_LOGITS_BF16 ? 16 : 32);
  const int lane = threadIdx.x & 31;
  OnlineSoftmax os;
  os.init(P.inv_t);
  raw_max = -INFINITY;
  raw_idx = -1;
  int raw_e = -1;  // first element of the stage in which this thread set the warp's maximum
  bool ok = true;

  // called by all lanes of the warp together
  auto consume = [&](const float (&l)[U][8], int e) {
    float vmax = max8(l[0]);
    if (U == 2) vmax = fmaxf(vmax, max8(l[U - 1]));
    const int wkey = __reduce_max_sync(0xffffffffu, ord_key(vmax));
    if (__builtin_expect(wkey > os.Mkey, 0)) {  // warp-uniform, rare
      const float wmax = ord_val(wkey);
      os.raise_to(wmax, wkey);
      if (vmax == wmax) {  // which element it was is looked up once, after the loop
        raw_max = wmax;
        raw_e = e;
      }
    }
#pragma unroll
    for (int g = 0; g < U; ++g) os.add8(l[g]);
  };
  // s = stage (a compile-time constant in the unrolled main loop), ph = parity of its current fill
  auto read_stage = [&](int s, uint32_t ph, float (&l)[U][8]) {
    ok = ok && mbar_wait_likely(full0 + 8 * s, ph, P.wait_ns);
    const uint32_t base = mine + s * kRowStageBytes;
#pragma unroll
    for (int g = 0; g < U; ++g) {
      uint4 a, b = make_uint4(0u, 0u, 0u, 0u);
      const uint32_t addr = base + g * (kRowStageBytes / U);
      asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w) : "r"(addr) : "memory");
      if (DT != ISD_LOGITS_BF16)
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w) : "r"(addr + 16) : "memory");
      unpack8<DT>(a, b, l[g]);
    }
    __syncwarp();
    if (lane == 0) ring_mbar_arrive(empty0 + 8 * s);  // the values are in registers: the stage may be refilled
  };

  // Stages in which every thread has all its data need no checks; the ragged last one is peeled.  The main
  // loop takes one trip round the ring per iteration, so stage numbers are constants and the parity flips
  // once per iteration.
  const int n = hi > lo ? hi - lo : 0;
  const int full = n / kStageElems;
  int e = lo + threadIdx.x * 8;
  int c = 0;
  uint32_t ph = 0;
  for (; c + kRowStages <= full; c += kRowStages, ph ^= 1) {
#pragma unroll
    for (int s = 0; s < kRowStages; ++s, e += kStageElems) {
      float l[U][8];
      read_stage(s, ph, l);
      consume(l, e);
    }
  }
  for (; c < full; ++c, e += kStageElems) {  // fewer than kRowStages left: stages 0, 1, ... of this round
    float l[U][8];
    read_stage(c & (kRowStages - 1), ph, l);
    consume(l, e);
  }
  if (full * kStageElems < n) {  // uniform over the CTA
    float l[U][8];
    read_stage(c & (kRowStages - 1), ph, l);
#pragma unroll
    for (int g = 0; g < U; ++g)
      if (!(e + g * kGroupStep < hi)) {
#pragma unroll
        for (int i = 0; i < 8; ++i) l[g][i] = -INFINITY;
      }
    consume(l, e);
  }
  if (raw_e >= 0) {
    // lowest index among this thread's elements of that stage that holds the recorded maximum
#pragma unroll
    for (int g = U - 1; g >= 0; --g) {
      const int eg = raw_e + g * kGroupStep;
      if (eg < hi) {
        float l[8];
        load8<DT>(row, eg, l);
#pragma unroll
        for (int i = 7; i >= 0; --i)
          if (l[i] == raw_max) raw_idx = eg + i;
      }
    }
  }
  S_out = os.sum();
  warp_max = os.M;  // the same in every lane
  return ok;
}

// A wait of the row pass ran out: the slot's statistics are incomplete, so the slot is marked (the decision
// phase and the commit then leave it alone) and the global word tells the host.
__device__ __forceinline__ void row_timeout(const VerifyParams& P, int b) {
  atomicOr(&P.slot_status[b], ISD_ST_KERNEL_TIMEOUT);
  atomicOr(P.global_status, ISD_ST_KERNEL_TIMEOUT);
}

// ------------------------------------------------------------------------------------------------
// Pass 1: row statistics
// ------------------------------------------------------------------------------------------------
template <int DT>
__device__ __forceinline__ void verify_rows_body(const VerifyParams& P, RowRing& sm_ring) {
  // Launch order = (split, slot, k): the rows that the sampling pass reads again come last, so that
  // they are the most recent lines in L2 when it starts.
  const int split = blockIdx.x, b = blockIdx.y, k = blockIdx.z;
  const int act = P.active[b];
  const int nv = P.n_ver[b];  // both loads in flight together
  if (!act) return;
  if (nv < 0 || nv > P.N - 1) {
    if (split == 0 && k == 0 && threadIdx.x == 0) {
      atomicOr(&P.slot_status[b], ISD_ST_SLOT_CAPACITY);
      atomicOr(P.global_status, ISD_ST_SLOT_CAPACITY);
    }
    return;
  }
  const int q_len = nv + P.N;
  int r = k + nv + rows_sampled(P);  // k = Q - rows_sampled .. Q - 1  <->  r = nv .. nv + rows_sampled - 1
  if (r >= P.Q) r -= P.Q;
  if (r >= q_len) return;

  const size_t elt = DT == ISD_LOGITS_BF16 ? 2 : 4;
  const char* row = reinterpret_cast<const char*>(P.logits_cur) + ((size_t)b * P.Q + r) * (size_t)P.V * elt;
  int lo, hi;
  chunk_range(P.V, P.row_splits, split, lo, hi);
  if (threadIdx.x >= kThreads) {
    // producer warp: one thread feeds the ring, then the warp is done (every copy it issued is consumed
    // by the workers before they leave; a wait that runs out raises the status bit and stops feeding)
    if (threadIdx.x == kThreads && hi > lo) {
      if (!row_producer(sm_ring, row, (size_t)lo * elt, (size_t)hi * elt, P.wait_ns)) row_timeout(P, b);
    }
    return;
  }

  float wmax, S, raw_max;
  int raw_idx;
  const bool ok = row_pass<DT>(P, sm_ring, row, lo, hi, wmax, S, raw_max, raw_idx);

  // ---- warp reduction -> partial, and the warp is done: one 16-byte store that nobody in this kernel reads.
  // Anything more at the end of a CTA (a CTA-wide merge, a fence and a ticket for a last-arriver decision)
  // keeps its share of the SM without a copy in flight for two or three round trips through a saturated memory
  // system, which at five CTAs per SM was an eighth of the kernel's time; the decision that needs all rows of
  // a slot is taken at the head of the sampling kernel instead.  Every lane of a warp holds the same maximum
  // (the warp agreed on it in every iteration), so its sums add up as they are, and the lowest index among the
  // lanes that recorded this maximum is the first occurrence in the warp's share.
  constexpr int kWarps = kThreads / 32;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) S += __shfl_xor_sync(0xffffffffu, S, off);
  const int widx = __reduce_min_sync(0xffffffffu, (raw_idx >= 0 && raw_max == wmax) ? raw_idx : 0x7FFFFFFF);
  if (lane == 0 && !ok) row_timeout(P, b);
  const float4 mine = make_float4(wmax * P.inv_t, S, wmax, __int_as_float(widx == 0x7FFFFFFF ? -1 : widx));
  float4* parts = reinterpret_cast<float4*>(P.row_part);
  if (P.row_splits == 1) {  // large batches: one partial per warp, see above
    if (lane == 0) parts[((size_t)b * P.Q + r) * kWarps + warp] = mine;
    return;
  }
  // Small batches cut a row into several CTAs and are bound by latency, not by copies in flight: one partial per
  // CTA keeps the merge at the head of the sampling kernel short.
  __shared__ float4 sm_part[kWarps];
  if (lane == 0) sm_part[warp] = mine;
  worker_sync();
  if (warp != 0) return;
  float4 v = lane < kWarps ? sm_part[lane] : make_float4(-INFINITY, 0.f, -INFINITY, __int_as_float(-1));
#pragma unroll
  for (int off = kWarps / 2; off > 0; off >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, v.x, off), os = __shfl_xor_sync(0xffffffffu, v.y, off);
    const float orw = __shfl_xor_sync(0xffffffffu, v.z, off);
    const int oi = __float_as_int(__shfl_xor_sync(0xffffffffu, v.w, off)), mi = __float_as_int(v.w);
    lse_merge(v.x, v.y, om, os);
    if (oi >= 0 && (mi < 0 || orw > v.z || (orw == v.z && oi < mi))) { v.z = orw; v.w = __int_as_float(oi); }
  }
  if (lane == 0) parts[((size_t)b * P.Q + r) * P.row_splits + split] = v;
}

// Inside isd_step the kernel before this one is the attention's combine kernel, of which the row pass needs
// nothing: what it reads - the step's logits and the slots' state - was complete and visible before the step's
// first kernel returned from its own wait.  There the pass starts streaming at once (rows_early), beside the
// last CTAs of the combine kernel, and waits for it only before it ends, which keeps the order of completion
// along the chain: the sampling kernel, whose last CTA rewrites the state the attention read, still cannot start
// before the attention is done.  On its own (isd_verify) the pass may follow the very kernel that wrote the
// logits, so it waits first.
template <int DT>
__global__ void __launch_bounds__(kThreads + 32, 5) verify_rows_kernel(const VerifyParams P) {
  __shared__ RowRing sm_ring;
  if (threadIdx.x == kThreads) {  // needs nothing from memory: runs while the kernel before this one drains
    for (int i = 0; i < kRowStages; ++i) {
      ring_mbar_init(ring_smem_u32(&sm_ring.full[i]), 1);
      ring_mbar_init(ring_smem_u32(&sm_ring.empty[i]), kThreads / 32);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();  // the only CTA-wide barrier of the kernel, still ahead of the wait
  if (!P.rows_early) pdl_wait();
  pdl_launch_dependents();
  verify_rows_body<DT>(P, sm_ring);
  if (P.rows_early) pdl_wait();
}

// ------------------------------------------------------------------------------------------------
// Pass 2: the random draws
// ------------------------------------------------------------------------------------------------
// fp64 score of vocabulary index i of the residual law: ln max(0, p_i - q_i) + g
__device__ double resid_score_f64(const VerifyParams& P, const void* prow, const void* qrow, int i, int x,
                                  double lse_p, double lse_q, uint32_t step, uint32_t slot, uint32_t tagpos) {
  const double pi = exp((double)load_logit(prow, P.logits_dtype, (size_t)i) * (double)P.inv_t - lse_p);
  double qi;
  if (P.q_mode == 0) qi = exp((double)load_logit(qrow, P.logits_dtype, (size_t)i) * (double)P.inv_t - lse_q);
  else qi = (i == x) ? 1.0 : 0.0;
  const double rres = pi - qi;
  if (!(rres > 0.0)) return -INFINITY;
  const uint4 r = philox4x32_10((uint32_t)i >> 2, step, slot, tagpos, P.seed_lo, P.seed_hi);
  return log(rres) + gumbel_f64(philox_word(r, i & 3));
}

// What one CTA of the sampling pass draws from.
struct SampleJob {
  const char* prow;  // the row whose law (or whose law minus q) is sampled
  const char* qrow;  // residual only, softmax q: the proposal-law row of the previous step
  int x;             // residual only: the rejected token
  float lse_p, lse_q;
  uint32_t tagpos;
  uint32_t step;     // Philox counter word of this step
  bool resid;
};

// fp32 noisy score of element i of the job's law; -inf when the element has no mass.  The same
// arithmetic scores the seed, the queued candidates and the fallback.
__device__ __forceinline__ float job_score(const VerifyParams& P, const SampleJob& J, float l, int i, uint32_t w) {
  if (!(l > -INFINITY)) return -INFINITY;
  if (!J.resid) return l * P.inv_t + gumbel_f32(w);
  const float pi = expf(l * P.inv_t - J.lse_p);
  const float qi = P.q_mode == 0 ? expf(load_logit(J.qrow, P.logits_dtype, (size_t)i) * P.inv_t - J.lse_q)
                                 : (i == J.x ? 1.f : 0.f);
  const float rr = pi - qi;
  return rr > 0.f ? logf(rr) + gumbel_f32(w) : -INFINITY;
}

// ------------------------------------------------------------------------------------------------
// Head of a sampling CTA, run by its warp 0: what the row pass found about the slot, the slot's decision
// (Algorithm 1, introspection loop) when the CTA draws the slot's emission (k = 0), the job of the CTA and the
// seed of its draw.  Every CTA takes the decision for itself; the one with split 0 records the slot's outputs
// that need no random sample (write).  Everything the head reads that does not depend on something else it
// reads is fetched in one go, so that the head costs two trips to memory (three for a residual against softmax q).
// ------------------------------------------------------------------------------------------------
struct SampleHead {
  int rej;        // -2: nothing for this CTA to draw (slot inactive or invalid; MASK row of a slot that makes no
                  // proposals); -1: frozen, nothing is drawn for the emission; 0: nothing rejected; j: first
                  // rejected proposal
  int nv;
  int r;          // row of this step's logits that the CTA draws from
  int x;          // residual: the rejected token
  int q_row;      // residual against softmax q: the row of q_prev that holds the proposal law
  float lse_p, lse_q;
  unsigned best;  // ordered code of the seed score (0: none)
};

constexpr int kHeadChunk = 8;  // partials of a row merged per pass (one pass unless the row pass cut a row into more than eight CTAs)

// Called by all 32 lanes of warp 0.  d_*: 32 entries of shared memory each.
template <int DT>
__device__ __forceinline__ void sample_head(const VerifyParams& P, int b, int k, int split, float* d_lse, float* d_raw,
                                            int* d_tok, int* d_bad, SampleHead* H) {
  const unsigned full = 0xffffffffu;
  const int lane = threadIdx.x & 31;
  const int NP = P.N - 1;
  const size_t elt = DT == ISD_LOGITS_BF16 ? 2 : 4;
  const size_t row_bytes = (size_t)P.V * elt;
  const char* cur = reinterpret_cast<const char*>(P.logits_cur) + (size_t)b * P.Q * row_bytes;
  const bool write = (k == 0 && split == 0);

  // ---- before the wait: the slots' state and the step's logits were complete before the kernel ahead of this one
  // could start (see verify_rows_kernel), so the proposals and their logits in the rows that judge them are
  // fetched while that kernel drains
  const int act = P.active[b];
  const int nv = P.n_ver[b];
  const bool is_pos = lane >= 1 && lane <= NP;  // lane = proposal position j (valid when j <= nv)
  int x = 0;
  float logq = 0.f, lse_q = 0.f;
  if (is_pos) {
    x = P.block_tok[(size_t)b * P.Q + lane];
    if (P.q_mode == 0) {
      const float* qs = P.q_stats + ((size_t)b * NP + lane - 1) * 2;
      lse_q = qs[0];
      logq = qs[1] - lse_q;
    }
  }
  const int q_row0 = (k == 0 && P.q_mode == 0) ? P.q_row0[b] : 0;
  const bool slot_ok = act && nv >= 0 && nv <= NP;  // an invalid n_ver was flagged by the row pass
  const bool pos = slot_ok && is_pos && lane <= nv;
  const bool badtok = pos && (x < 0 || x >= P.V);
  float lx = 0.f;  // the raw logit of the proposal in the row that judges it
  if (pos && !badtok) lx = load_logit(cur + (size_t)(lane - 1) * row_bytes, P.logits_dtype, (size_t)x);

  pdl_wait();
  // ---- after it: what the row pass wrote, in one trip
  const int n_part = P.row_splits == 1 ? kThreads / 32 : P.row_splits;  // per warp of the row's CTA, or per CTA
  const bool has_row = lane < P.Q;  // lane = block row (rows beyond the slot's block hold stale partials, unused)
  const float4* rp = reinterpret_cast<const float4*>(P.row_part) + ((size_t)b * P.Q + (has_row ? lane : 0)) * n_part;
  const float4 neutral = make_float4(-INFINITY, 0.f, -INFINITY, __int_as_float(-1));
  float4 part[kHeadChunk];
#pragma unroll
  for (int i = 0; i < kHeadChunk; ++i) part[i] = i < n_part ? __ldcg(rp + i) : neutral;
  // a warp of the row pass gave up on a wait: a partial is incomplete, nothing of the slot may be committed
  const uint32_t timeout = *reinterpret_cast<volatile uint32_t*>(&P.slot_status[b]) & ISD_ST_KERNEL_TIMEOUT;

  if (!slot_ok) {
    if (lane == 0) H->rej = -2;
    return;
  }
  const int q_len = nv + P.N;

  {  // lane = block row: merge its partials (max and sum of the online softmax, first argmax)
    float m = -INFINITY, s = 0.f, best = -INFINITY;
    int tok = -1;
    for (int c = 0;; ) {
      float cm = -INFINITY;
#pragma unroll
      for (int i = 0; i < kHeadChunk; ++i) {
        const int id = __float_as_int(part[i].w);
        cm = fmaxf(cm, part[i].x);
        if (id >= 0 && (part[i].z > best || (part[i].z == best && id < tok) || tok < 0)) { best = part[i].z; tok = id; }
      }
      const float nm = fmaxf(m, cm);
      if (nm > -INFINITY) {
        float acc = (m > -INFINITY) ? s * __expf(m - nm) : 0.f;
#pragma unroll
        for (int i = 0; i < kHeadChunk; ++i)
          if (part[i].x > -INFINITY) acc += part[i].y * __expf(part[i].x - nm);  // NaN sums and m = +inf poison s
        s = acc;
      }
      m = nm;
      c += kHeadChunk;
      if (c >= n_part) break;
#pragma unroll
      for (int i = 0; i < kHeadChunk; ++i) part[i] = c + i < n_part ? __ldcg(rp + c + i) : neutral;
    }
    const bool valid = lane < q_len;
    // NaN anywhere poisons s; +inf logits give m = +inf
    d_bad[lane] = valid && ((s != s) || (m == INFINITY) || (m != m));
    d_lse[lane] = m + logf(s);
    d_raw[lane] = best;
    d_tok[lane] = valid ? tok : -1;
  }
  __syncwarp();

  int rej = 0, a = nv;
  bool frozen = false;
  {
    // The accept tests of all positions at once (a test depends on nothing an earlier one decides); the first
    // position that rejects, or whose token id is out of range, ends the sequence.
    float al = NAN;
    bool acc = true;
    if (pos && !badtok) {
      const float logp = lx * P.inv_t - d_lse[lane - 1];
      al = (1.f + P.tau) * expf(logp - logq);
      al = fminf(al, 1.f);
      if (al != al) al = 0.f;
      const uint4 rnd = philox4x32_10(0u, step_of(P), (uint32_t)b, (ISD_TAG_ACCEPT << 16) | (uint32_t)lane, P.seed_lo, P.seed_hi);
      const float u = (float)(rnd.x >> 8) * 0x1p-24f;
      acc = u < al;
    }
    const unsigned m_badtok = __ballot_sync(full, badtok);
    const unsigned m_stop = m_badtok | __ballot_sync(full, pos && !badtok && !acc);
    const int first = m_stop ? __ffs(m_stop) - 1 : nv + 1;
    const bool bad_first = m_stop && ((m_badtok >> first) & 1u);
    rej = (m_stop && !bad_first) ? first : 0;
    a = bad_first ? -1 : (rej ? rej - 1 : nv);
    const bool evald = pos && lane <= first && !badtok;  // positions whose test was run
    const bool nonfinite = (evald && d_bad[lane - 1]) || (lane >= 1 && lane <= NP && d_bad[nv + lane]) ||
                           (lane == 0 && a >= 0 && rej == 0 && d_bad[nv]);
    uint32_t status = timeout;
    if (__ballot_sync(full, nonfinite)) status |= ISD_ST_NONFINITE_LOGIT;
    if (bad_first) status |= ISD_ST_BAD_TOKEN_ID;
    frozen = a < 0 || (status & ~ISD_ST_EMPTY_RESIDUAL);
    const int x_next = __shfl_down_sync(full, x, 1);  // lane j - 1 gets proposal j
    // the rejected token and the LSE of its proposal law, for the residual
    const int x_rej = __shfl_sync(full, x, rej);
    const float lse_q_rej = __shfl_sync(full, lse_q, rej);
    if (lane == 0) {
      H->x = x_rej;
      H->lse_q = lse_q_rej;
    }

    if (write) {
      if (lane >= 1 && lane <= NP) {
        P.out.accept[(size_t)b * NP + lane - 1] = evald ? (lane == rej ? 0 : 1) : -1;
        P.out.alpha[(size_t)b * NP + lane - 1] = evald ? al : NAN;
        // Proposals of the MASK rows (lanes 1..N-1 = MASK row m) and their law's statistics.  After a rejection
        // the rows were conditioned on discarded tokens and the next step is a pure stride step (Sec. 3.2): no
        // proposals are made.  Argmax proposals are final here; sampled ones and their logit are written by the
        // CTAs that draw them.
        const bool proposes = !frozen && rej == 0;
        const int rr = nv + lane;
        P.out.new_q_stats[((size_t)b * NP + lane - 1) * 2 + 0] = proposes ? d_lse[rr] : NAN;
        if (P.propose_mode == 1 || !proposes) {
          const int xh = proposes ? d_tok[rr] : -1;
          P.out.new_prop_tok[(size_t)b * NP + lane - 1] = xh;
          // the raw logit at the first argmax is the row's maximum
          P.out.new_q_stats[((size_t)b * NP + lane - 1) * 2 + 1] = xh >= 0 ? d_raw[rr] * P.inv_t : NAN;
        }
      }
      // the emission: accepted proposals now; the drawn token and the copy of it in repl_tok come from the CTA
      // of the sampling pass that finishes the draw, unless nothing is drawn
      const bool draws = !frozen && !(rej > 0 && P.q_mode == 0 && P.q_prev == nullptr);
      if (lane < P.N && !(draws && lane == a))
        P.out.out_tok[(size_t)b * P.N + lane] = (!frozen && lane < a) ? x_next : -1;
      if (lane == 0) {
        if (!draws) P.out.repl_tok[b] = -1;
        P.out.accept_len[b] = frozen ? 0 : a;
        P.out.n_emit[b] = frozen ? 0 : a + 1;
        if (frozen) {
          atomicOr(&P.slot_status[b], status);
          atomicOr(P.global_status, status);
        }
      }
    }
  }
  if (lane != 0) return;

  // ---- the CTA's job and the seed of its draw: the true noisy score of the row's argmax, whose raw logit is the
  // row's maximum (for the residual: if it has residual mass)
  H->nv = nv;
  H->rej = frozen ? -1 : rej;
  if (k > 0 && (frozen || rej != 0)) {  // a MASK row of a slot that makes no proposals
    H->rej = -2;
    return;
  }
  const int r = (k == 0 && rej > 0) ? rej - 1 : nv + k;
  H->r = r;
  H->q_row = q_row0 + rej - 1;
  H->lse_p = rej > 0 ? d_lse[rej - 1] : 0.f;
  H->best = 0u;
  if (frozen) return;
  SampleJob J;
  J.resid = k == 0 && rej > 0;
  J.x = H->x; J.lse_p = H->lse_p; J.lse_q = H->lse_q;
  J.qrow = nullptr;
  if (J.resid && P.q_mode == 0) {
    if (P.q_prev == nullptr) return;  // nothing to subtract: nothing is drawn
    J.qrow = reinterpret_cast<const char*>(P.q_prev) + ((size_t)b * P.Q + H->q_row) * row_bytes;
  }
  J.step = step_of(P);
  J.tagpos = k == 0 ? ((ISD_TAG_FINAL << 16) | (uint32_t)(rej > 0 ? rej : nv + 1)) : ((ISD_TAG_PROPOSE << 16) | (uint32_t)k);
  const int i0 = d_tok[r];
  if (i0 >= 0 && i0 < P.V) {
    const uint4 rnd = philox4x32_10((uint32_t)i0 >> 2, J.step, (uint32_t)b, J.tagpos, P.seed_lo, P.seed_hi);
    const float seed = job_score(P, J, d_raw[r], i0, philox_word(rnd, i0 & 3));
    if (seed > -INFINITY) H->best = enc_ordered(seed);
  }
}

// resident CTAs per SM the sampling kernel is compiled for: three keep it at 80 registers (without the bound
// the compiler takes 89 and only two CTAs fit)
constexpr int kSampleMinBlocks = 4;
// Per-warp queue of groups of four logits that survived the first skip test.
constexpr int kQueueCap = 128;  // < 32 left over + at most 64 new per iteration
struct SampleQueue {
  float4 l[kThreads / 32][kQueueCap];
  int idx[kThreads / 32][kQueueCap];
};

// Gumbel-max top-2 of elements [lo, hi) of the job's law.  `best` enters as a noisy score that some
// element of the row really has (the seed, or -inf), so it is a lower bound of the winner's score; it is
// shared by the CTA through sm_best, and a stale value only makes the skip tests weaker.
template <int DT>
__device__ __forceinline__ void sample_pass(const VerifyParams& P, const SampleJob& J, int lo, int hi, int b,
                                            float best, Top2& top, SampleQueue& Q, unsigned* sm_best,
                                            RowStream<DT, 1, kSampleRingBytes>& in) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned below = (1u << lane) - 1u;
  float4* ql = Q.l[warp];
  int* qi = Q.idx[warp];
  const float scale2 = P.inv_t * kLog2e;
  const float rcp_t = 1.f / P.inv_t;
  // the law's log-mass of element i is at most l_i invT - shift (residual: ln r_i <= ln p_i)
  const float shift = J.resid ? J.lse_p : 0.f;
  const float cut_off = (shift - kGumbelMax) * rcp_t;
  top.init();
  int head = 0, tail = 0;  // warp-uniform queue positions

  // Judge one queued group whose noise `rnd` has been drawn, and keep its candidates.
  auto judge = [&](int idx, const float4& v, const uint4& rnd) {
    // -ln u' >= 1 - u' >= nf 2^-24 with nf = floor(2^24 (1 - u')) = (~word) >> 8, so g_i <= -ln(nf 2^-24): element i
    // cannot come within 2e-3 of the running best when nf >= 1.002 * 2^24 * exp(l_i invT - shift - best).
    // First for the whole group, with the group's largest logit and in integers: nf >= kb for the integer
    // kb >= that bound is the same as word <= ~(kb << 8), one compare per element and no conversion.  Nearly
    // every group ends here.
    float K2 = 24.0028853901f - (shift + best) * kLog2e;  // log2 of the factor; +inf while there is no best
    const float xg = fmaf(fmaxf(max3(v.x, v.y, v.z), v.w), scale2, K2);
    if (xg < 23.9f) {  // false for NaN (no best yet) and for groups that reach the running best
      uint32_t kb;
      asm("cvt.rpi.u32.f32 %0, %1;" : "=r"(kb) : "f"(ex2f(xg)));
      const uint32_t wt = ~(kb << 8);
      if (rnd.x <= wt && rnd.y <= wt && rnd.z <= wt && rnd.w <= wt) return;
    }
    const float l4[4] = {v.x, v.y, v.z, v.w};
    const uint32_t w[4] = {rnd.x, rnd.y, rnd.z, rnd.w};
    bool improved = false;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float nf = (float)((~w[i]) >> 8);
      const float bound = ex2f(fmaf(l4[i], scale2, K2));
      if (!(nf >= bound)) {
        const float sc = job_score(P, J, l4[i], idx + i, w[i]);
        if (sc > -INFINITY) {
          top.push(sc, idx + i);
          if (top.s1 > best) {
            best = top.s1;
            K2 = 24.0028853901f - (shift + best) * kLog2e;
            improved = true;
          }
        }
      }
    }
    if (improved) atomicMax(sm_best, enc_ordered(best));
  };
  auto drain = [&](int pos) {
    const int idx = qi[pos & (kQueueCap - 1)];
    const float4 v = ql[pos & (kQueueCap - 1)];
    const uint4 rnd = philox4x32_10((uint32_t)idx >> 2, J.step, (uint32_t)b, J.tagpos, P.rk);
    judge(idx, v, rnd);
  };

  // uniform trip count per block (the warp votes inside the loop)
  for (int base = lo; base < hi; base += kThreads * 8) {
    const int e = base + threadIdx.x * 8;
    float lg[1][8];
    in.next(lg);
    float (&l)[8] = lg[0];
    if (!(e < hi)) {
#pragma unroll
      for (int i = 0; i < 8; ++i) l[i] = -INFINITY;
    }
    best = fmaxf(best, dec_ordered(*reinterpret_cast<volatile unsigned*>(sm_best)));
    const float cut = fmaf(best, rcp_t, cut_off);  // raw-logit units; -inf while there is no best
    const float g0 = fmaxf(fmaxf(l[0], l[1]), fmaxf(l[2], l[3]));
    const float g1 = fmaxf(fmaxf(l[4], l[5]), fmaxf(l[6], l[7]));
    const bool p0 = g0 > cut, p1 = g1 > cut;  // false for padding and all -inf groups
    const unsigned m0 = __ballot_sync(0xffffffffu, p0);
    const unsigned m1 = __ballot_sync(0xffffffffu, p1);
    if (p0) {
      const int s = (tail + __popc(m0 & below)) & (kQueueCap - 1);
      ql[s] = make_float4(l[0], l[1], l[2], l[3]);
      qi[s] = e;
    }
    tail += __popc(m0);
    if (p1) {
      const int s = (tail + __popc(m1 & below)) & (kQueueCap - 1);
      ql[s] = make_float4(l[4], l[5], l[6], l[7]);
      qi[s] = e + 4;
    }
    tail += __popc(m1);
    __syncwarp();
    while (tail - head >= 32) {
      drain(head + lane);
      head += 32;
    }
  }
  in.finish();
  __syncwarp();
  if (lane < tail - head) drain(head + lane);
}

// Returns whether this CTA is the one that reports its (slot, k) to the step's ticket: the last of the CTAs that
// drew for it, or the one with split 0 when none of them has anything to draw.
template <int DT>
__device__ __forceinline__ bool verify_sample_body(const VerifyParams& P) {
  const int split = blockIdx.x, k = blockIdx.y, b = blockIdx.z;

  __shared__ float sm_f0[kThreads / 32], sm_f1[kThreads / 32];
  __shared__ int sm_i0[kThreads / 32], sm_i1[kThreads / 32];
  __shared__ int sm_last, sm_tok;
  __shared__ unsigned sm_best;
  __shared__ SampleQueue sm_queue;
  __shared__ __align__(16) uint4 sm_ring[kSampleRingBytes / 16];
  __shared__ float d_lse[32], d_raw[32];
  __shared__ int d_tok[32], d_bad[32];
  __shared__ SampleHead sm_head;

  // ---- what the row pass found, the slot's decision, this CTA's job and its seed (the other warps wait)
  if (threadIdx.x < 32) {
    sample_head<DT>(P, b, k, split, d_lse, d_raw, d_tok, d_bad, &sm_head);  // executes the wait
    if (threadIdx.x == 0) sm_best = sm_head.rej >= 0 ? sm_head.best : 0u;
  } else {
    pdl_wait();
  }
  __syncthreads();
  const int rej = sm_head.rej;
  if (rej == -2) return split == 0;             // inactive or invalid slot, or no proposals to draw
  if (k == 0 && rej < 0) return split == 0;     // frozen slot: no emission
  const int nv = sm_head.nv;

  const int NP = P.N - 1;
  const size_t elt = DT == ISD_LOGITS_BF16 ? 2 : 4;
  const size_t row_bytes = (size_t)P.V * elt;
  const char* cur = reinterpret_cast<const char*>(P.logits_cur) + (size_t)b * P.Q * row_bytes;

  // ---- what this (slot, k) draws
  SampleJob J;
  J.qrow = nullptr; J.x = -1; J.lse_p = 0.f; J.lse_q = 0.f;
  J.step = step_of(P);
  const int r = sm_head.r;  // row of this step's logits that is sampled
  if (k == 0 && rej > 0) {
    // replacement for the first rejected proposal, from normalize(max(0, p - q))
    if (P.q_mode == 0 && P.q_prev == nullptr) return split == 0;  // nothing to subtract: the caller gave no proposal-law rows
    J.resid = true;
    J.x = sm_head.x;
    J.lse_p = sm_head.lse_p;
    if (P.q_mode == 0) {
      J.qrow = reinterpret_cast<const char*>(P.q_prev) + ((size_t)b * P.Q + sm_head.q_row) * row_bytes;
      J.lse_q = sm_head.lse_q;
    }
    J.tagpos = (ISD_TAG_FINAL << 16) | (uint32_t)rej;
  } else {
    // k = 0: bonus / free token from the row of the last clean token; k >= 1: MASK row k
    J.resid = false;
    J.tagpos = k == 0 ? ((ISD_TAG_FINAL << 16) | (uint32_t)(nv + 1)) : ((ISD_TAG_PROPOSE << 16) | (uint32_t)k);
  }
  J.prow = cur + (size_t)r * row_bytes;

  int lo, hi;
  chunk_range(P.V, P.sample_splits, split, lo, hi);
  RowStream<DT, 1, kSampleRingBytes> in;
  in.start(sm_ring, J.prow, lo, hi);
  const float best0 = dec_ordered(sm_best);  // NaN when there is no seed

  Top2 top;
  sample_pass<DT>(P, J, lo, hi, b, fmaxf(-INFINITY, best0), top, sm_queue, &sm_best, in);

  block_merge_top2(top, sm_f0, sm_i0, sm_f1, sm_i1);
  int* ticket = P.samp_ticket + (size_t)b * P.N + k;
  SamplePartial* parts = P.samp_part + ((size_t)b * P.N + k) * P.sample_splits;
  if (threadIdx.x == 0) {
    SamplePartial sp;
    sp.best1 = top.s1; sp.idx1 = top.i1; sp.best2 = top.s2; sp.idx2 = top.i2;
    parts[split] = sp;
    __threadfence();
    const int arrived = atomicAdd(ticket, 1);
    sm_last = (arrived == P.sample_splits - 1);
  }
  __syncthreads();
  if (!sm_last) return false;
  __threadfence();

  // ---- last CTA of the (slot, k): merge, fp64 tie-break, write the token
  if (threadIdx.x < 32) {
    Top2 t;
    t.init();
    if ((int)threadIdx.x < P.sample_splits) {  // at most 16 pieces: one per lane
      const volatile SamplePartial* sp = parts + threadIdx.x;
      t.s1 = sp->best1; t.i1 = sp->idx1; t.s2 = sp->best2; t.i2 = sp->idx2;
    }
    warp_top2(t);
    if (threadIdx.x == 0) {
      *ticket = 0;  // ready for the next call
      int y = t.i1;
      if (t.i1 >= 0 && t.i2 >= 0 && (t.s1 - t.s2) < ISD_TIE_EPS) {
        double s1, s2;
        if (J.resid) {
          s1 = resid_score_f64(P, J.prow, J.qrow, t.i1, J.x, J.lse_p, J.lse_q, J.step, (uint32_t)b, J.tagpos);
          s2 = resid_score_f64(P, J.prow, J.qrow, t.i2, J.x, J.lse_p, J.lse_q, J.step, (uint32_t)b, J.tagpos);
        } else {
          s1 = noisy_score_f64(P, J.prow, t.i1, J.step, (uint32_t)b, J.tagpos);
          s2 = noisy_score_f64(P, J.prow, t.i2, J.step, (uint32_t)b, J.tagpos);
        }
        if (s2 > s1 || (s2 == s1 && t.i2 < t.i1)) y = t.i2;
      }
      sm_tok = y;
    }
  }
  __syncthreads();
  int y = sm_tok;
  if (J.resid && y < 0) {
    // Residual empty in fp32 (p and q numerically equal): fall back to a sample of p with the same
    // noise.  Rare; done by this one CTA over the whole row.
    J.resid = false;
    if (threadIdx.x == 0) sm_best = 0u;
    __syncthreads();
    Top2 t;
    in.start(sm_ring, J.prow, 0, P.V);
    sample_pass<DT>(P, J, 0, P.V, b, -INFINITY, t, sm_queue, &sm_best, in);
    block_merge_top2(t, sm_f0, sm_i0, sm_f1, sm_i1);
    if (threadIdx.x == 0) {
      y = t.i1;
      if (t.i1 >= 0 && t.i2 >= 0 && (t.s1 - t.s2) < ISD_TIE_EPS) {
        const double s1 = noisy_score_f64(P, J.prow, t.i1, J.step, (uint32_t)b, J.tagpos);
        const double s2 = noisy_score_f64(P, J.prow, t.i2, J.step, (uint32_t)b, J.tagpos);
        if (s2 > s1 || (s2 == s1 && t.i2 < t.i1)) y = t.i2;
      }
      atomicOr(&P.slot_status[b], ISD_ST_EMPTY_RESIDUAL);
      atomicOr(P.global_status, ISD_ST_EMPTY_RESIDUAL);
    }
  }
  if (threadIdx.x == 0) {
    if (k == 0) {
      const int a = rej > 0 ? rej - 1 : nv;
      P.out.repl_tok[b] = y;
      P.out.out_tok[(size_t)b * P.N + a] = y;
    } else {
      P.out.new_prop_tok[(size_t)b * NP + k - 1] = y;
      P.out.new_q_stats[((size_t)b * NP + k - 1) * 2 + 1] =
          y >= 0 ? load_logit(J.prow, P.logits_dtype, (size_t)y) * P.inv_t : NAN;
    }
  }
  return true;
}

template <int DT>
__global__ void __launch_bounds__(kThreads, kSampleMinBlocks) verify_sample_kernel(const VerifyParams P) {
  pdl_launch_dependents();
  const bool reports = verify_sample_body<DT>(P);  // executes griddepcontrol.wait after its first loads
  if (!P.fuse_commit || !reports) return;
  // ---- isd_step: every (slot, k) is reported once to a ticket over the grid, after its token is written; the
  // CTA that reports last (nobody waits) has every slot's decision and tokens in front of it and commits the
  // batch, which saves the launch of a kernel for it
  __shared__ int sm_commit[36];
  if (threadIdx.x == 0) {
    __threadfence();  // what this CTA wrote (tokens, status bits) comes before its report
    const int arrived = atomicAdd(P.step_ticket, 1);
    sm_commit[35] = (arrived == (int)(gridDim.y * gridDim.z) - 1);
  }
  __syncthreads();
  if (!sm_commit[35]) return;
  if (threadIdx.x == 0) *P.step_ticket = 0;  // ready for the next call
  __threadfence();
  commit_block(P.commit, sm_commit, sm_commit + 33);
}

}  // namespace

// CTAs a row of the row pass is cut into: enough CTAs to fill the machine (five per SM run at once) at small
// batch, one CTA per row once rows are plentiful; a piece keeps at least 8k elements.
int isd_pick_row_splits(const isd_config& c, int num_sms) {
  const int rows = c.batch * (2 * c.stride - 1);
  const int max_by_len = (c.vocab + 8191) / 8192;
  int rs = (4 * num_sms + rows - 1) / rows;
  rs = rs < 1 ? 1 : (rs > 16 ? 16 : rs);
  return rs > max_by_len ? max_by_len : rs;
}

// Pieces a sampled row is cut into.  Large batches: four (every further piece starts again from the seed alone
// and re-learns the running best; eight cost 45 % more work on flat rows).  Small batches are latency-bound and
// leave most SMs idle, so their rows are cut finer, up to sixteen pieces, as long as all CTAs are resident at once
// (four per SM; batch 1: 50 -> 42 us of verification).
int isd_pick_sample_splits(const isd_config& c, int num_sms) {
  const int rows = c.batch * (c.propose_mode == 0 ? c.stride : 1);
  const int max_by_len = (c.vocab + 8191) / 8192;  // keep at least 8k elements per CTA
  int ps = 4 * num_sms / rows;  // rounded down: a few CTAs more than the SMs hold at once would double the pass
  ps = ps < 4 ? 4 : (ps > 16 ? 16 : ps);
  return ps > max_by_len ? max_by_len : ps;
}

int isd_launch_verify(isd_ctx* ctx, const isd_batch_state* st, const void* logits_cur,
                      const void* q_prev_logits, uint32_t step, const isd_verify_out* out,
                      cudaStream_t stream, isd_batch_state* commit_st) {
  const isd_config& c = ctx->cfg;
  VerifyParams P;
  P.B = c.batch; P.N = c.stride; P.Q = ctx->Q; P.V = c.vocab;
  P.logits_dtype = c.logits_dtype; P.q_mode = c.q_mode; P.propose_mode = c.propose_mode;
  P.inv_t = c.inv_temperature; P.tau = c.tau;
  P.wait_ns = ctx->wait_ns;
  philox_round_keys(c.seed, P.rk);
  P.seed_lo = (uint32_t)c.seed; P.seed_hi = (uint32_t)(c.seed >> 32); P.step = step;
  P.step_dev = ctx->step_counter;
  P.row_splits = ctx->row_splits; P.sample_splits = ctx->sample_splits;
  P.n_ver = st->n_ver; P.active = st->active; P.block_tok = st->block_tok; P.q_row0 = st->q_row0;
  P.q_stats = st->q_stats; P.slot_status = st->slot_status; P.global_status = ctx->global_status;
  P.logits_cur = logits_cur; P.q_prev = q_prev_logits; P.out = *out;
  P.row_part = ctx->row_part; P.samp_part = ctx->samp_part; P.samp_ticket = ctx->samp_ticket;
  P.fuse_commit = commit_st != nullptr && ctx->step_ticket != nullptr;
  P.rows_early = commit_st != nullptr;  // called from isd_step / isd_step_layers, behind the step's attention
  P.step_ticket = ctx->step_ticket;
  P.commit = make_commit_params(ctx, P.fuse_commit ? commit_st : st, out);

  const dim3 grid1(ctx->row_splits, c.batch, ctx->Q);
  const dim3 grid2(ctx->sample_splits, c.propose_mode == 0 ? c.stride : 1, c.batch);
  if (ctx->ev_verify0) cudaEventRecord(ctx->ev_verify0, stream);
  cudaError_t e1, e2;
  if (c.logits_dtype == ISD_LOGITS_BF16) {
    e1 = isd_launch_pdl(verify_rows_kernel<ISD_LOGITS_BF16>, grid1, dim3(kThreads + 32), 0, stream, P);
    e2 = isd_launch_pdl(verify_sample_kernel<ISD_LOGITS_BF16>, grid2, dim3(kThreads), 0, stream, P);
  } else {
    e1 = isd_launch_pdl(verify_rows_kernel<ISD_LOGITS_F32>, grid1, dim3(kThreads + 32), 0, stream, P);
    e2 = isd_launch_pdl(verify_sample_kernel<ISD_LOGITS_F32>, grid2, dim3(kThreads), 0, stream, P);
  }
  if (ctx->ev_verify1) cudaEventRecord(ctx->ev_verify1, stream);
  ctx->launches += 2;
  if (e1 != cudaSuccess || e2 != cudaSuccess) return ISD_ERR_CUDA;
  // without the fused commit the caller launches the commit kernel itself
  return ISD_OK;
}

// ------------------------------------------------------------------------------------------------
// isd_verify_static: the same two verification kernels, for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the point where they verify: a serving
// engine that has handed every free byte of the device to its own KV-cache allocator, a runtime
// that forbids allocation on its latency-critical thread, or code that runs while another component
// holds the allocator.  isd_create (which owns the scratch of isd_verify) is closed to them.  For
// those callers the scratch lives in the fixed device array below, which every GPU that loads the
// library keeps until the process exits, and the entry point touches neither cudaMalloc/cudaFree
// nor any allocating library routine.
//
// Capacity: at most ISD_STATIC_MAX_BATCH slots (any stride the library supports).  Larger batches
// are refused with ISD_ERR_TOO_LARGE before anything is launched.
// ------------------------------------------------------------------------------------------------
#include <mutex>

namespace {

constexpr int kStaticMaxBatch = ISD_STATIC_MAX_BATCH;
constexpr int kStaticMaxSplits = 16;
constexpr size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }
// layout of the array: [zeroed every call: tickets of the sampling pass, status word][partials of both passes]
constexpr int kStaticMaxStride = (ISD_MAX_Q + 1) / 2;
constexpr size_t kOffSampTicket = 0;
constexpr size_t kOffStatus = kOffSampTicket + align256(sizeof(int) * kStaticMaxBatch * kStaticMaxStride);
constexpr size_t kZeroedBytes = kOffStatus + align256(sizeof(uint32_t));
constexpr size_t kOffSampPart = kZeroedBytes;
constexpr size_t kOffRowPart =
    kOffSampPart + align256(sizeof(SamplePartial) * kStaticMaxBatch * kStaticMaxStride * kStaticMaxSplits);
// row pieces of one call: rows * row_splits <= rows + 4 * SMs by the rule that picks row_splits; the entry point
// lowers row_splits where a device with more SMs would exceed this.  One partial per worker warp of a piece.
constexpr int kStaticMaxRowPieces = kStaticMaxBatch * ISD_MAX_Q + 1024;
constexpr size_t kStaticBytes = kOffRowPart + align256(sizeof(RowPartial) * kStaticMaxRowPieces * (kThreads / 32));

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
unsigned char* g_static_ptr[kMaxDevices] = {};

}  // namespace

// File-scope device array (about 0.65 MB per GPU).  In host code this name is only a handle for
// cudaGetSymbolAddress; it is never passed to a kernel directly.
static __device__ __align__(256) unsigned char g_isd_verify_static_scratch[kStaticBytes];

extern "C" int isd_verify_static(const isd_config* cfg, const isd_batch_state* st, const void* logits_cur,
                                 const void* q_prev_logits, uint64_t step, const isd_verify_out* out,
                                 void* cuda_stream) {
  if (!cfg || !st || !out || !logits_cur || step > 0xFFFFFFFFull) return ISD_ERR_INVALID_ARG;
  const isd_config& c = *cfg;
  if (c.batch < 1 || c.stride < 1 || c.vocab < 8 || c.inv_temperature <= 0.f || c.tau < 0.f) return ISD_ERR_INVALID_ARG;
  if (c.logits_dtype != ISD_LOGITS_F32 && c.logits_dtype != ISD_LOGITS_BF16) return ISD_ERR_INVALID_ARG;
  if (c.q_mode < 0 || c.q_mode > 1 || c.propose_mode < 0 || c.propose_mode > 1) return ISD_ERR_INVALID_ARG;
  if (2 * c.stride - 1 > ISD_MAX_Q || c.vocab % 8 != 0 || c.top_k != 0) return ISD_ERR_UNSUPPORTED;
  if (c.batch > kStaticMaxBatch) return ISD_ERR_TOO_LARGE;
  if (!st->n_ver || !st->active || !st->block_tok || !st->q_row0 || !st->slot_status) return ISD_ERR_INVALID_ARG;
  if (c.stride > 1 && (!st->q_stats || !out->accept || !out->alpha || !out->new_prop_tok || !out->new_q_stats))
    return ISD_ERR_INVALID_ARG;
  if (!out->accept_len || !out->n_emit || !out->repl_tok || !out->out_tok) return ISD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(logits_cur) & 15u) || (reinterpret_cast<uintptr_t>(q_prev_logits) & 15u))
    return ISD_ERR_ALIGNMENT;

  // one-time set-up per device: resolve the device address of the scratch array with that device current
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ISD_ERR_CUDA;
  unsigned char* base = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_isd_verify_static_scratch) != cudaSuccess || !p) return ISD_ERR_CUDA;
      g_static_ptr[dev] = static_cast<unsigned char*>(p);
    }
    base = g_static_ptr[dev];
  }

  // a context on the host stack that points into the static array; nothing is allocated
  isd_ctx tmp = {};
  tmp.cfg = c;
  tmp.device = dev;
  tmp.Q = 2 * c.stride - 1;
  tmp.G = 1;
  int sms = 0;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  tmp.num_sms = sms > 0 ? sms : ISD_NUM_SMS_DEFAULT;
  const int rows = c.batch * tmp.Q;
  int rs = isd_pick_row_splits(c, tmp.num_sms);  // <= kStaticMaxSplits
  if (rows * rs > kStaticMaxRowPieces) rs = kStaticMaxRowPieces / rows;  // >= 1: rows <= 64 * ISD_MAX_Q
  tmp.row_splits = rs;
  tmp.sample_splits = isd_pick_sample_splits(c, tmp.num_sms);  // same cut as isd_create uses (<= kStaticMaxSplits)
  tmp.samp_ticket = reinterpret_cast<int*>(base + kOffSampTicket);
  tmp.global_status = reinterpret_cast<uint32_t*>(base + kOffStatus);
  tmp.samp_part = reinterpret_cast<SamplePartial*>(base + kOffSampPart);
  tmp.row_part = reinterpret_cast<RowPartial*>(base + kOffRowPart);
  tmp.wait_ns = ISD_DEFAULT_WAIT_NS;

  // the array keeps the previous call's contents: counters and flags must start at zero
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(base, 0, kZeroedBytes, stream) != cudaSuccess) return ISD_ERR_CUDA;
  return isd_launch_verify(&tmp, st, logits_cur, q_prev_logits, (uint32_t)step, out, stream);
}

extern "C" int isd_test_verify_grid(const isd_config* cfg, int32_t num_sms, int32_t* out) {
  if (!cfg || !out || num_sms < 1 || cfg->batch < 1 || cfg->stride < 1 || cfg->vocab < 8) return ISD_ERR_INVALID_ARG;
  const isd_config& c = *cfg;
  const int rs = isd_pick_row_splits(c, num_sms), ps = isd_pick_sample_splits(c, num_sms);
  out[0] = rs;
  out[1] = ps;
  out[2] = rs * c.batch * (2 * c.stride - 1);
  out[3] = ps * c.batch * (c.propose_mode == 0 ? c.stride : 1);
  return ISD_OK;
}
