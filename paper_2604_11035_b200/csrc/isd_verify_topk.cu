// isd_verify on top-k / top-p filtered laws (the serving sampling configuration of the paper's
// appendix: temperature, top-k = 50, top-p = 0.95).  Algorithm 1 is applied to the filtered,
// renormalised laws: F(row) keeps the top_k entries in the order (value descending, index
// ascending) and of those the shortest prefix whose probability mass reaches top_p.
//
// With at most ISD_MAX_TOP_K tokens of support per law, everything after the selection is tiny, and
// no vocabulary-wide exponentials are needed at all:
//   1. topk_rows_kernel    one CTA per (slot, block row): the exact top-k of the row in one stream of
//      it (block_topk).  Per logit: a packed maximum over groups of eight and one compare against a
//      rising bound; the few groups that reach it are re-read from L2 and ranked.  The CTA that
//      finishes a slot's last row runs the rest of the slot: nucleus cut and log-normaliser of every
//      row in fp64 (the oracle's arithmetic, so the cut agrees), the sequential accept test, and the
//      Gumbel-max draws (residual, bonus, proposals) over the supports in fp64 with the same
//      per-index Philox noise as the unfiltered path.  The filtered proposal law a rejection needs
//      is a list of the previous call (kept by the context) whenever q_prev_logits is that call's
//      buffer: then this is the only kernel.
//   2. topk_decide_kernel  otherwise: one cluster of kQSplit CTAs per slot with a rejection selects
//      the top-k of the proposal-law row again, one piece per CTA, and the first CTA merges the
//      pieces and draws the replacement.
#include "isd_internal.cuh"
#include "isd_stream.cuh"
#include "isd_commit.cuh"

#include <cooperative_groups.h>

namespace {

constexpr int kMaxTopK = ISD_MAX_TOP_K;
constexpr int kCandCap = 1024;  // candidate keys in shared memory
constexpr int kGroupCap = 512;  // queued groups in shared memory
constexpr int kQSplit = 2;      // CTAs (one cluster) per slot in the decide kernel: pieces of a proposal-law row

struct TopkParams {
  int B, N, Q, V;
  int logits_dtype, q_mode, propose_mode, top_k;
  float inv_t, tau, top_p;
  unsigned long long wait_ns;  // time limit of a device-side wait
  uint32_t seed_lo, seed_hi, step;
  const uint32_t* step_dev;
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
  float* list_val;  // [B, Q, kMaxTopK] raw logits of the row's top-k, best first
  int* list_idx;    // [B, Q, kMaxTopK]
  int* list_n;      // [B, Q] entries of the list; -1 - n when the row holds a NaN or +inf
  // the same three of the previous call (read only), valid when q_prev is the row buffer that call selected from
  const float* prev_val;
  const int* prev_idx;
  const int* prev_n;
  int prev_valid;
  unsigned long long* q_key;  // [B, kQSplit, kMaxTopK] piece lists of the proposal-law row of a rejection
  int* q_n;                   // [B, kQSplit]
  int* q_dec;                 // [B, 2] accept length (-1: frozen) and rejected position, from the row kernel to the decide kernel
  int* nuc_n;                 // [B, Q] support size of every row's filtered law
  int* nuc_bad;               // [B, Q] 1 = the row holds a NaN or +inf
  double* nuc_lse;            // [B, Q] log-normaliser of the support
  int* row_ticket;            // [B] rows of the slot that are done (zero between launches)
  // isd_step: the CTA of the row kernel that finishes last commits the batch (fuse_commit != 0)
  int fuse_commit;
  int rows_early;  // isd_step: the row kernel starts before the kernel ahead of it has completed (see topk_rows_kernel)
  int* step_ticket;
  CommitParams commit;
};

struct TopkShared {
  RowRing ring;
  __align__(16) unsigned long long key[kCandCap];
  unsigned long long sorted[kMaxTopK];
  unsigned offer[kThreads / 32];
  int group[kGroupCap];  // first element of every group of eight that may hold a candidate
  int count, gcount, bad, again, have, over;
  float list_val[kMaxTopK];
  int list_idx[kMaxTopK];
  int list_n;
};

// Larger key = better candidate: higher value first, lower index on equal values.
__device__ __forceinline__ unsigned value_key(float v) { return (unsigned)ord_key(v) ^ 0x80000000u; }
__device__ __forceinline__ unsigned long long cand_key(float v, int idx) {
  return ((unsigned long long)value_key(v) << 32) | (unsigned long long)(0xFFFFFFFFu - (unsigned)idx);
}
__device__ __forceinline__ float key_value(unsigned long long k) { return ord_val((int)((unsigned)(k >> 32) ^ 0x80000000u)); }
__device__ __forceinline__ int key_index(unsigned long long k) { return (int)(0xFFFFFFFFu - (unsigned)k); }

__device__ __forceinline__ float max_nan(float a, float b) {  // NaN if either is NaN
  float d;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
  return d;
}

// Appends the elements of a group of eight that reach the bound.  Deliberately not inlined: the call keeps this
// rare path (about one group in three hundred) behind a real branch; inlined, the compiler predicates it and
// every group pays for its instructions.
__device__ __noinline__ void collect_group(TopkShared* sh, float x0, float x1, float x2, float x3, float x4, float x5,
                                           float x6, float x7, int e, unsigned long long bound) {
  const float x[8] = {x0, x1, x2, x3, x4, x5, x6, x7};
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    if (x[i] > -INFINITY) {
      const unsigned long long kk = cand_key(x[i], e + i);
      if (kk >= bound) {
        const int pos = atomicAdd(&sh->count, 1);
        if (pos < kCandCap) sh->key[pos] = kk;
      }
    }
  }
}

// The largest of the eight logits of a group, NaN if one of them is NaN.  bf16 pairs are compared packed: three
// two-lane maxima, then the two halves of the last word.  (Which of -0 and +0 wins is irrelevant to the callers:
// they use the result in float comparisons, or as a lower bound.)
template <int DT>
__device__ __forceinline__ float group_max(const uint4& a, const uint4& b) {
  if (DT == ISD_LOGITS_BF16) {
    uint32_t m0, m1, m;
    asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(m0) : "r"(a.x), "r"(a.y));
    asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(m1) : "r"(a.z), "r"(a.w));
    asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(m) : "r"(m0), "r"(m1));
    return max_nan(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u));
  }
  const float m0 = max_nan(max_nan(__uint_as_float(a.x), __uint_as_float(a.y)), max_nan(__uint_as_float(a.z), __uint_as_float(a.w)));
  const float m1 = max_nan(max_nan(__uint_as_float(b.x), __uint_as_float(b.y)), max_nan(__uint_as_float(b.z), __uint_as_float(b.w)));
  return max_nan(m0, m1);
}

// Sorts key[0, n) descending (bitonic, padded with zeros to a power of two <= kCandCap).  Worker threads only.
__device__ void sort_keys(unsigned long long* key, int n) {
  int m = 2;
  while (m < n) m <<= 1;
  for (int i = n + threadIdx.x; i < m; i += kThreads) key[i] = 0ull;  // padding sorts last
  worker_sync();
  for (int size = 2; size <= m; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int t = threadIdx.x; t < (m >> 1); t += kThreads) {
        const int lo = 2 * t - (t & (stride - 1));
        const int hi = lo + stride;
        const bool desc = ((lo & size) == 0);
        const unsigned long long a = key[lo], b = key[hi];
        if ((a < b) == desc) { key[lo] = b; key[hi] = a; }
      }
      worker_sync();
    }
  }
}

// The best k of n <= kThreads distinct non-zero keys, best first, by counting: thread t ranks key t among all of
// them (no barriers inside, unlike a sorting network).  Result in out[0, return value).  Worker threads only.
__device__ int rank_select(const unsigned long long* key, int n, int k, unsigned long long* out) {
  if (threadIdx.x < n) {
    const unsigned long long mine = key[threadIdx.x];
    int r0 = 0, r1 = 0;
    int j = 0;
    for (; j + 4 <= n; j += 4) {  // key is 16-byte aligned: two keys per load
      const ulonglong2 p = *reinterpret_cast<const ulonglong2*>(key + j);
      const ulonglong2 q = *reinterpret_cast<const ulonglong2*>(key + j + 2);
      r0 += (p.x > mine ? 1 : 0) + (q.x > mine ? 1 : 0);
      r1 += (p.y > mine ? 1 : 0) + (q.y > mine ? 1 : 0);
    }
    for (; j < n; ++j) r0 += key[j] > mine ? 1 : 0;
    if (r0 + r1 < k) out[r0 + r1] = mine;
  }
  worker_sync();
  return n < k ? n : k;
}

// A value that at least k elements reach, from the threads' maxima, without a block-wide sort: every warp sorts
// its 32 maxima with shuffles and offers its ceil(k / warps)-th best; the smallest offer is reached by that many
// maxima in every warp, k or more in all.  0 when some warp has too few finite maxima (then everything finite is
// collected).  Worker threads only.
__device__ unsigned bound_from_maxima(unsigned vkey, int k, unsigned* sm_offer) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned v = vkey;
#pragma unroll
  for (int size = 2; size <= 32; size <<= 1) {
#pragma unroll
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      const unsigned o = __shfl_xor_sync(0xffffffffu, v, stride);
      const bool up = ((lane & size) == 0), lower = ((lane & stride) == 0);
      v = (lower == up) ? (v > o ? v : o) : (v < o ? v : o);
    }
  }
  const int per_warp = (k + kThreads / 32 - 1) / (kThreads / 32);
  if (lane == per_warp - 1) sm_offer[warp] = v;  // descending: lane r - 1 holds the r-th best
  worker_sync();
  unsigned b = sm_offer[0];
#pragma unroll
  for (int w = 1; w < kThreads / 32; ++w) b = b < sm_offer[w] ? b : sm_offer[w];
  return b;
}

// Exact top-k of a whole logits row, by all kThreads + 32 threads of the CTA: leaves the list (best first)
// in sh.list_* / sh.list_n and the non-finite flag in sh.bad.  Returns false when a wait ran out.
//
// The row is streamed twice.  First stream: every thread keeps the best value it sees, and from those maxima
// comes a value that at least k elements of the row reach, i.e. a lower bound of the row's k-th best (a tight
// one: the top-k fall into mostly distinct threads).  Second stream: every element that reaches the bound is
// collected, about k plus a few dozen, and ranked by (value, index).  Should the collected set overflow the
// buffer (many equal values), the k-th best of what was collected is a strictly better bound and the second
// stream is repeated.
template <int DT>
__device__ bool block_topk_two_stream(TopkShared& sh, const char* row, int e_lo, int e_hi, int k, unsigned long long wait_ns) {
  constexpr int kElt = DT == ISD_LOGITS_BF16 ? 2 : 4;
  constexpr int U = DT == ISD_LOGITS_BF16 ? 2 : 1;
  constexpr int kStageElems = kRowStageBytes / kElt;
  constexpr int kGroupStep = kStageElems / U;
  const bool worker = threadIdx.x < kThreads;
  const uint32_t full0 = ring_smem_u32(sh.ring.full), empty0 = ring_smem_u32(sh.ring.empty);
  const uint32_t mine = ring_smem_u32(sh.ring.stage) + threadIdx.x * (DT == ISD_LOGITS_BF16 ? 16 : 32);
  const int lane = threadIdx.x & 31;
  const int stages = (e_hi - e_lo + kStageElems - 1) / kStageElems;
  bool ok = true;
  unsigned long long bound = 0ull;
  if (threadIdx.x == 0) sh.bad = 0;
  for (int pass = 0;; ++pass) {
    if (threadIdx.x == 0) {
      for (int i = 0; i < kRowStages; ++i) {
        ring_mbar_init(ring_smem_u32(&sh.ring.full[i]), 1);
        ring_mbar_init(ring_smem_u32(&sh.ring.empty[i]), kThreads / 32);
      }
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      sh.count = 0;
      sh.again = 0;
    }
    __syncthreads();
    if (!worker) {
      if (threadIdx.x == kThreads) ok = row_producer(sh.ring, row, (size_t)e_lo * kElt, (size_t)e_hi * kElt, wait_ns) && ok;
    } else {
      float tmax = -INFINITY;  // first stream: the best value this thread has seen
      int e = e_lo + threadIdx.x * 8;
      for (int c = 0; c < stages; ++c, e += kStageElems) {
        const int s = c & (kRowStages - 1);
        ok = mbar_wait_likely(full0 + 8 * s, (uint32_t)(c / kRowStages) & 1u, wait_ns) && ok;
        float l[U][8];
#pragma unroll
        for (int g = 0; g < U; ++g) {
          uint4 a, b = make_uint4(0u, 0u, 0u, 0u);
          const uint32_t addr = mine + s * kRowStageBytes + g * (kRowStageBytes / U);
          asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w) : "r"(addr) : "memory");
          if (DT != ISD_LOGITS_BF16)
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w) : "r"(addr + 16) : "memory");
          unpack8<DT>(a, b, l[g]);
          if (c == stages - 1 && !(e + g * kGroupStep < e_hi)) {  // beyond the range
#pragma unroll
            for (int i = 0; i < 8; ++i) l[g][i] = -INFINITY;
          }
        }
        __syncwarp();
        if (lane == 0) ring_mbar_arrive(empty0 + 8 * s);
#pragma unroll
        for (int g = 0; g < U; ++g) {
          const float gmax = max_nan(max_nan(max_nan(l[g][0], l[g][1]), max_nan(l[g][2], l[g][3])),
                                     max_nan(max_nan(l[g][4], l[g][5]), max_nan(l[g][6], l[g][7])));
          if (gmax != gmax || gmax == INFINITY) {
            sh.bad = 1;  // NaN or +inf somewhere in the eight: the slot will be frozen, the list does not matter
            continue;
          }
          if (pass == 0) {
            tmax = fmaxf(tmax, gmax);  // value only: which element it was does not matter for a bound
          } else if (gmax > -INFINITY && value_key(gmax) >= (unsigned)(bound >> 32)) {
            collect_group(&sh, l[g][0], l[g][1], l[g][2], l[g][3], l[g][4], l[g][5], l[g][6], l[g][7],
                          e + g * kGroupStep, bound);
          }
        }
      }
      if (pass == 0) {
        bound = (unsigned long long)bound_from_maxima(tmax > -INFINITY ? value_key(tmax) : 0u, k, sh.offer) << 32;
        if (threadIdx.x == 0) sh.again = 1;
      } else {
        worker_sync();
        const int total = sh.count;
        worker_sync();  // everybody has read the count
        int n;
        if (total <= kThreads) {  // the usual case
          n = rank_select(sh.key, total, k, sh.sorted);
        } else {
          const int collected = total < kCandCap ? total : kCandCap;
          sort_keys(sh.key, collected);
          n = collected < k ? collected : k;
          if (threadIdx.x < n) sh.sorted[threadIdx.x] = sh.key[threadIdx.x];
          if (total > kCandCap && pass < 4096) {  // overflow (many equal values): a strictly better bound, once more
            bound = sh.key[k - 1];
            if (threadIdx.x == 0) sh.again = 1;
          }
          worker_sync();
        }
        if (threadIdx.x < n) {
          sh.list_val[threadIdx.x] = key_value(sh.sorted[threadIdx.x]);
          sh.list_idx[threadIdx.x] = key_index(sh.sorted[threadIdx.x]);
        }
        if (threadIdx.x == 0) sh.list_n = n;
      }
    }
    __syncthreads();  // producer warp and workers meet; sh.again is final
    if (!sh.again) break;
    __syncthreads();  // everybody has read the flag before thread 0 clears it for the next pass
  }
  return ok;
}

constexpr int kHeadStages = 8;  // stages of the head, read twice to find a first bound
constexpr int kCheckEvery = 8;  // stages between two looks at the queue of noted groups (a power of two)
constexpr int kExpandAt = 64;   // noted groups from which a look turns them into candidates
constexpr int kCompactAt = 96;  // candidates from which they are cut back to the best k and the bound rises

// One stage of the ring: waits for it, takes this thread's groups of eight as packed words, releases the stage.
template <int DT, int U>
__device__ __forceinline__ bool take_stage(uint32_t full0, uint32_t empty0, uint32_t mine, int cc, uint4 (&a)[U], uint4 (&b)[U],
                                           unsigned long long wait_ns) {
  const int s = cc & (kRowStages - 1);
  const bool ok = mbar_wait_likely(full0 + 8 * s, (uint32_t)(cc / kRowStages) & 1u, wait_ns);
#pragma unroll
  for (int g = 0; g < U; ++g) {
    b[g] = make_uint4(0u, 0u, 0u, 0u);
    const uint32_t addr = mine + s * kRowStageBytes + g * (kRowStageBytes / U);
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(a[g].x), "=r"(a[g].y), "=r"(a[g].z), "=r"(a[g].w) : "r"(addr) : "memory");
    if (DT != ISD_LOGITS_BF16)
      asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(b[g].x), "=r"(b[g].y), "=r"(b[g].z), "=r"(b[g].w) : "r"(addr + 16) : "memory");
  }
  __syncwarp();
  if ((threadIdx.x & 31) == 0) ring_mbar_arrive(empty0 + 8 * s);
  return ok;
}

// Exact top-k of elements [e_lo, e_hi) of a logits row (e_lo a multiple of 8) in ONE stream of them (plus their
// head a second time), by all kThreads + 32 threads of the CTA; same result as block_topk_two_stream: the list
// (best first) in sh.list_* / sh.list_n and the non-finite flag in sh.bad.  Returns false when a wait ran out.
//
// The head (kHeadStages stages) goes through the ring first: the threads' maxima over it give a value that k of
// its elements reach.  Then the whole range follows through the same ring, head included (those bytes come from
// L2).  The common path per group of eight is its packed maximum and one compare.  A group whose maximum reaches
// the bound is only noted (its element index goes to a queue).  At the end of the head, and then every
// kCheckEvery stages, the workers look at the queue; when it is long enough they expand it densely, one group
// per thread, re-reading the eight logits from global memory (L2): the elements that reach the bound become
// candidates, and from kCompactAt candidates on the best k are kept and the bound rises to the k-th best so
// far, so that fewer and fewer groups are noted (about k ln(n / head) after the head).  When more arrives
// between two looks than the buffers hold (a row sorted upwards, long runs of equal values), nothing more is
// noted, the stream is drained and the two-stream routine, which handles any input, starts over.
template <int DT>
__device__ bool block_topk(TopkShared& sh, const char* row, int e_lo, int e_hi, int k, unsigned long long wait_ns) {
  constexpr int kElt = DT == ISD_LOGITS_BF16 ? 2 : 4;
  constexpr int U = DT == ISD_LOGITS_BF16 ? 2 : 1;
  constexpr int kStageElems = kRowStageBytes / kElt;
  constexpr int kGroupStep = kStageElems / U;
  const bool worker = threadIdx.x < kThreads;
  const int stages = (e_hi - e_lo + kStageElems - 1) / kStageElems;
  // the head: kHeadStages stages of a long range, a quarter of a short one (it is read twice)
  const int head = stages >= 4 * kHeadStages ? kHeadStages : stages >= 4 ? stages / 4 : stages > 0 ? 1 : 0;
  bool ok = true;
  if (threadIdx.x == 0) {
    for (int i = 0; i < kRowStages; ++i) {
      ring_mbar_init(ring_smem_u32(&sh.ring.full[i]), 1);
      ring_mbar_init(ring_smem_u32(&sh.ring.empty[i]), kThreads / 32);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    sh.count = 0;
    sh.gcount = 0;
    sh.bad = 0;
    sh.over = 0;
    sh.list_n = 0;
  }
  __syncthreads();
  if (!worker) {
    if (threadIdx.x == kThreads) {
      const size_t lo = (size_t)e_lo * kElt, hi = (size_t)e_hi * kElt, head_hi = lo + (size_t)head * kRowStageBytes;
      int c = 0;
      ok = row_producer(sh.ring, row, lo, head_hi < hi ? head_hi : hi, c, wait_ns);
      ok = ok && row_producer(sh.ring, row, lo, hi, c, wait_ns);
    }
  } else {
    const uint32_t full0 = ring_smem_u32(sh.ring.full), empty0 = ring_smem_u32(sh.ring.empty);
    const uint32_t mine = ring_smem_u32(sh.ring.stage) + threadIdx.x * (DT == ISD_LOGITS_BF16 ? 16 : 32);
    uint4 a[U], b[U];
    // ---- the head: the best value this thread sees
    float tmax = -INFINITY;
    for (int c = 0; c < head; ++c) {
      ok = take_stage<DT, U>(full0, empty0, mine, c, a, b, wait_ns) && ok;
      const int e = e_lo + c * kStageElems + threadIdx.x * 8;
#pragma unroll
      for (int g = 0; g < U; ++g) {
        if (c == stages - 1 && !(e + g * kGroupStep < e_hi)) continue;  // beyond the range
        const float gmax = group_max<DT>(a[g], b[g]);
        if (gmax < INFINITY) tmax = fmaxf(tmax, gmax);  // value only: which element it was does not matter for a bound
      }
    }
    // candidates are the keys >= bound; a group is noted when its maximum reaches the bound's value
    unsigned long long bound = (unsigned long long)bound_from_maxima(tmax > -INFINITY ? value_key(tmax) : 0u, k, sh.offer) << 32;
    float bound_f = bound ? key_value(bound) : -INFINITY;
    bool over = false;
    // ---- the range
    for (int c = 0; c < stages; ++c) {
      ok = take_stage<DT, U>(full0, empty0, mine, head + c, a, b, wait_ns) && ok;
      const int e = e_lo + c * kStageElems + threadIdx.x * 8;
      const bool last = c == stages - 1;
#pragma unroll
      for (int g = 0; g < U; ++g) {
        const bool valid = !last || e + g * kGroupStep < e_hi;
        const float gmax = group_max<DT>(a[g], b[g]);
        const bool finite = gmax < INFINITY;  // false for NaN too
        if (__any_sync(0xffffffffu, valid && (!finite || gmax >= bound_f))) {  // rare for the warp as a whole
          if (valid && !finite) {
            sh.bad = 1;  // NaN or +inf somewhere in the eight: the slot will be frozen, the list does not matter
          } else if (valid && gmax >= bound_f) {
            const int pos = atomicAdd(&sh.gcount, 1);
            if (pos < kGroupCap) sh.group[pos] = e + g * kGroupStep;
          }
        }
      }
      const bool head_end = c == head - 1;
      if (!last && !head_end && (c & (kCheckEvery - 1)) != kCheckEvery - 1) continue;
      // ---- a look at the queue
      worker_sync();
      const int groups = sh.gcount;
      if (groups > kGroupCap) {  // too much between two looks: note nothing more, start over below
        over = true;
        bound_f = INFINITY;
        continue;  // (the count stays above the capacity, so every later look ends here as well)
      }
      if (!last && !head_end && groups < kExpandAt) {
        worker_sync();  // everybody has read the count before anybody adds to it
        continue;
      }
      for (int i = threadIdx.x; i < groups; i += kThreads) {  // one group per thread, re-read from global memory
        const int ge = sh.group[i];
        float x[8];
        load8<DT>(row, ge, x);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (x[j] > -INFINITY) {
            const unsigned long long kk = cand_key(x[j], ge + j);
            if (kk >= bound) {
              const int pos = atomicAdd(&sh.count, 1);
              if (pos < kCandCap) sh.key[pos] = kk;
            }
          }
        }
      }
      worker_sync();
      const int total = sh.count;
      if (threadIdx.x == 0) sh.gcount = total > kCandCap ? kGroupCap + 1 : 0;  // overflow: as above
      worker_sync();  // everybody has read the counts; the queue is empty again
      if (total > kCandCap) {
        over = true;
        bound_f = INFINITY;
        continue;
      }
      if (!last && !head_end && total < kCompactAt) continue;
      int n;
      if (total <= kThreads) {  // the usual case
        n = rank_select(sh.key, total, k, sh.sorted);
      } else {
        sort_keys(sh.key, total);
        n = total < k ? total : k;
        if (threadIdx.x < n) sh.sorted[threadIdx.x] = sh.key[threadIdx.x];
        worker_sync();
      }
      if (last) {
        if (threadIdx.x < n) {
          sh.list_val[threadIdx.x] = key_value(sh.sorted[threadIdx.x]);
          sh.list_idx[threadIdx.x] = key_index(sh.sorted[threadIdx.x]);
        }
        if (threadIdx.x == 0) sh.list_n = n;
      } else {
        if (threadIdx.x < n) sh.key[threadIdx.x] = sh.sorted[threadIdx.x];
        if (threadIdx.x == 0) sh.count = n;
        if (n == k) {
          bound = sh.sorted[k - 1];
          bound_f = key_value(bound);
        }
        worker_sync();  // the cut-back buffer and its count are in place before the next look
      }
    }
    if (over && threadIdx.x == 0) sh.over = 1;
  }
  __syncthreads();  // producer warp and workers meet
  if (sh.over) return block_topk_two_stream<DT>(sh, row, e_lo, e_hi, k, wait_ns) && ok;
  return ok;
}

// Shared memory of the accept phase (it reuses the ring of a CTA whose row is done).
struct SlotScratch {
  int n[32], bad[32], x[32];
  float logp[32], logq[32];
  double lse[32];
  double w[kThreads / 32][kMaxTopK];
  int a, rej;  // accept length (-1: frozen) and rejected position (0: none)
};
static_assert(sizeof(SlotScratch) <= sizeof(RowRing::stage), "the accept phase lives in the ring's stages");

__device__ __forceinline__ float ldcg_f(const float* p) { return __ldcg(p); }
__device__ __forceinline__ int ldcg_i(const int* p) { return __ldcg(p); }

// Nucleus of a sorted top-k list in fp64, in the oracle's order of operations: w_i = exp(l_i invT - l_0 invT),
// Z = sum w_i, support = shortest prefix whose cumulated w reaches top_p * Z.  Returns the support size and
// the log-normaliser of the support.  By one warp: the lanes compute the exponentials (w: n doubles of shared
// memory), lane 0 adds them up in index order; every lane gets the result.  FROM_L2: the list is in global memory
// and is read from L2 (other CTAs of this launch may have written it).
template <bool FROM_L2>
__device__ int warp_nucleus(const float* val, int n, double inv_t, double top_p, double* w, double& lse) {
  const int lane = threadIdx.x & 31;
  lse = -INFINITY;
  if (n <= 0) return 0;
  const double m = (double)(FROM_L2 ? ldcg_f(val) : val[0]) * inv_t;
  if (isinf(m) && m < 0) return n;
  for (int i = lane; i < n; i += 32) w[i] = exp((double)(FROM_L2 ? ldcg_f(val + i) : val[i]) * inv_t - m);
  __syncwarp();
  // lane 0 adds in index order, once: w[i] becomes the sum of the first i + 1 (the oracle's three loops - the
  // normaliser, the cumulated mass, the mass of the support - add the same numbers in the same order)
  if (lane == 0) {
    double cum = 0.0;
    for (int i = 0; i < n; ++i) {
      cum += w[i];
      w[i] = cum;
    }
  }
  __syncwarp();
  const double Z = w[n - 1];
  int keep = n;
  for (int i0 = 0; i0 < n; i0 += 32) {
    const unsigned hit = __ballot_sync(0xffffffffu, i0 + lane < n && w[i0 + lane] >= top_p * Z);
    if (hit) { keep = i0 + __ffs(hit); break; }
  }
  const double l = m + log(w[keep - 1]);
  lse = l;
  __syncwarp();  // w may be reused
  return keep;
}

// The accept phase of one slot, by the CTA that finished the slot's last row (all its threads): support and
// log-normaliser of every row, then the sequential accept test (Algorithm 1, introspection loop) on the filtered
// laws.  Leaves the supports, the decision and the outputs that need no random draw in global memory.
__device__ void slot_accept(const TopkParams& P, SlotScratch& S, int b, int nv) {
  const int q_len = nv + P.N, NP = P.N - 1;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const double inv_t = (double)P.inv_t, top_p = (double)P.top_p;
  const uint32_t step = P.step_dev ? *P.step_dev : P.step;
  const float* LV = P.list_val + (size_t)b * P.Q * kMaxTopK;
  const int* LI = P.list_idx + (size_t)b * P.Q * kMaxTopK;
  // ---- every row's support and log-normaliser (one warp per row, rows dealt round-robin)
  if (warp < kThreads / 32) {
    for (int rr = warp; rr < q_len; rr += kThreads / 32) {
      int ln = ldcg_i(P.list_n + (size_t)b * P.Q + rr), bad = 0;
      if (ln < 0) { bad = 1; ln = -1 - ln; }
      double lse;
      const int n = warp_nucleus<true>(LV + (size_t)rr * kMaxTopK, ln, inv_t, top_p, S.w[warp], lse);
      if (lane == 0) {
        S.n[rr] = n; S.bad[rr] = bad; S.lse[rr] = lse;
        P.nuc_n[(size_t)b * P.Q + rr] = n; P.nuc_bad[(size_t)b * P.Q + rr] = bad; P.nuc_lse[(size_t)b * P.Q + rr] = lse;
      }
      // the inputs of the accept test at position rr + 1, whose anchor law this row is: the proposal, log p~ of it
      // (-inf unless it is in the support) and log q~ of it
      const int j = rr + 1;
      if (j <= nv) {
        const int x = P.block_tok[(size_t)b * P.Q + j];
        float logp = -INFINITY;
        for (int i = lane; i < n; i += 32)
          if (ldcg_i(LI + (size_t)rr * kMaxTopK + i) == x) logp = ldcg_f(LV + (size_t)rr * kMaxTopK + i) * P.inv_t - (float)lse;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) logp = fmaxf(logp, __shfl_xor_sync(0xffffffffu, logp, off));  // at most one lane found it
        if (lane == 0) {
          S.x[j] = x;
          S.logp[j] = logp;
          float logq = 0.f;
          if (P.q_mode == 0) {
            const float* qs = P.q_stats + ((size_t)b * NP + j - 1) * 2;
            logq = qs[1] - qs[0];
          }
          S.logq[j] = logq;
        }
      }
    }
  }
  __syncthreads();
  // ---- sequential accept test
  if (threadIdx.x == 0) {
    uint32_t status = 0;
    int a = nv, rej = 0;
    for (int m = 1; m <= NP; ++m) status |= S.bad[nv + m] ? ISD_ST_NONFINITE_LOGIT : 0u;
    for (int j = 1; j <= NP; ++j) {
      P.out.accept[(size_t)b * NP + j - 1] = -1;
      P.out.alpha[(size_t)b * NP + j - 1] = NAN;
    }
    for (int j = 1; j <= nv; ++j) {
      const int x = S.x[j];
      if (x < 0 || x >= P.V) { status |= ISD_ST_BAD_TOKEN_ID; a = -1; break; }
      if (S.bad[j - 1]) status |= ISD_ST_NONFINITE_LOGIT;
      const float logp = S.logp[j], logq = S.logq[j];
      float al = (1.f + P.tau) * expf(logp - logq);
      al = fminf(al, 1.f);
      if (al != al) al = 0.f;
      const uint4 rnd = philox4x32_10(0u, step, (uint32_t)b, (ISD_TAG_ACCEPT << 16) | (uint32_t)j, P.seed_lo, P.seed_hi);
      const float u = (float)(rnd.x >> 8) * 0x1p-24f;
      P.out.alpha[(size_t)b * NP + j - 1] = al;
      if (u < al) {
        P.out.accept[(size_t)b * NP + j - 1] = 1;
      } else {
        P.out.accept[(size_t)b * NP + j - 1] = 0;
        a = j - 1;
        rej = j;
        break;
      }
    }
    if (a >= 0 && rej == 0 && S.bad[nv]) status |= ISD_ST_NONFINITE_LOGIT;
    for (int j = 0; j < P.N; ++j) P.out.out_tok[(size_t)b * P.N + j] = -1;
    P.out.repl_tok[b] = -1;
    if (a < 0 || (status & ~ISD_ST_EMPTY_RESIDUAL)) {
      P.out.accept_len[b] = 0;
      P.out.n_emit[b] = 0;
      atomicOr(&P.slot_status[b], status);
      atomicOr(P.global_status, status);
      a = -1;
    } else {
      P.out.accept_len[b] = a;
      P.out.n_emit[b] = a + 1;
      for (int j = 1; j <= a; ++j) P.out.out_tok[(size_t)b * P.N + j - 1] = P.block_tok[(size_t)b * P.Q + j];
    }
    P.q_dec[2 * b] = a;
    P.q_dec[2 * b + 1] = rej;
    S.a = a;
    S.rej = rej;
  }
  __syncthreads();
}

// warp-wide arg max of (score, index): highest score, lowest index on ties (the oracle scans indices upwards
// and replaces only on a strictly greater score)
__device__ __forceinline__ void warp_argmax(double& s, int& idx) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const double os = __shfl_xor_sync(0xffffffffu, s, off);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, off);
    if (oi >= 0 && (idx < 0 || os > s || (os == s && oi < idx))) { s = os; idx = oi; }
  }
}

__device__ __forceinline__ double gumbel_at(const TopkParams& P, uint32_t step, int b, uint32_t tagpos, int idx) {
  const uint4 r = philox4x32_10((uint32_t)idx >> 2, step, (uint32_t)b, tagpos, P.seed_lo, P.seed_hi);
  return gumbel_f64(philox_word(r, idx & 3));
}

// The draws of a slot, once its supports (s_n, s_lse) and its accept decision are known.  The lists are read from
// L2: in the row kernel other CTAs of the same launch have written them.
//
// Proposals of the MASK rows: Gumbel-max over the support (warp m - 1 draws row nv + m), or its head.
// After a rejection (or on a frozen slot) the MASK rows were conditioned on discarded tokens: no proposals are made
// (Sec. 3.2: the next step is a pure stride step) and the outputs are set to -1 / NaN (used = false).
__device__ void draw_proposals(const TopkParams& P, const int* s_n, const double* s_lse, int b, int nv, uint32_t step, bool used) {
  const int NP = P.N - 1, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const double inv_t = (double)P.inv_t;
  const float* LV = P.list_val + (size_t)b * P.Q * kMaxTopK;
  const int* LI = P.list_idx + (size_t)b * P.Q * kMaxTopK;
  if (warp < 1 || warp >= kThreads / 32) return;
  for (int m = warp; m <= NP; m += kThreads / 32 - 1) {
    const int rr = nv + m, n = s_n[rr];
    const float* v = LV + (size_t)rr * kMaxTopK;
    const int* ix = LI + (size_t)rr * kMaxTopK;
    double best = -INFINITY;
    int tok = -1;
    float ltok = NAN;
    if (!used) {
      if (lane == 0) {
        P.out.new_prop_tok[(size_t)b * NP + m - 1] = -1;
        P.out.new_q_stats[((size_t)b * NP + m - 1) * 2 + 0] = NAN;
        P.out.new_q_stats[((size_t)b * NP + m - 1) * 2 + 1] = NAN;
      }
      continue;
    }
    if (P.propose_mode == 1) {
      if (n > 0) tok = ldcg_i(ix);
    } else {
      const uint32_t tagpos = (ISD_TAG_PROPOSE << 16) | (uint32_t)m;
      for (int i = lane; i < n; i += 32) {
        const double lp = (double)ldcg_f(v + i) * inv_t;
        if (isinf(lp) && lp < 0) continue;
        const int id = ldcg_i(ix + i);
        const double sc = lp + gumbel_at(P, step, b, tagpos, id);
        if (tok < 0 || sc > best || (sc == best && id < tok)) { best = sc; tok = id; }
      }
      warp_argmax(best, tok);
    }
    if (lane == 0) {
      for (int i = 0; i < n; ++i)
        if (ldcg_i(ix + i) == tok) ltok = ldcg_f(v + i) * P.inv_t;
      P.out.new_prop_tok[(size_t)b * NP + m - 1] = tok;
      P.out.new_q_stats[((size_t)b * NP + m - 1) * 2 + 0] = (float)s_lse[rr];
      P.out.new_q_stats[((size_t)b * NP + m - 1) * 2 + 1] = tok >= 0 ? ltok : NAN;
    }
  }
}

// Bonus / free token: Gumbel-max over the support of the row of the last clean token (warp 0).
__device__ void draw_bonus(const TopkParams& P, const int* s_n, int b, int nv, int a, uint32_t step) {
  const int lane = threadIdx.x & 31;
  if (threadIdx.x >= 32) return;
  const double inv_t = (double)P.inv_t;
  const int n = s_n[nv];
  const float* v = P.list_val + ((size_t)b * P.Q + nv) * kMaxTopK;
  const int* ix = P.list_idx + ((size_t)b * P.Q + nv) * kMaxTopK;
  const uint32_t tagpos = (ISD_TAG_FINAL << 16) | (uint32_t)(nv + 1);
  double best = -INFINITY;
  int tok = -1;
  for (int i = lane; i < n; i += 32) {
    const double lp = (double)ldcg_f(v + i) * inv_t;
    if (isinf(lp) && lp < 0) continue;
    const int id = ldcg_i(ix + i);
    const double sc = lp + gumbel_at(P, step, b, tagpos, id);
    if (tok < 0 || sc > best || (sc == best && id < tok)) { best = sc; tok = id; }
  }
  warp_argmax(best, tok);
  if (lane == 0) {
    P.out.repl_tok[b] = tok;
    P.out.out_tok[(size_t)b * P.N + a] = tok;
  }
}

// Replacement from normalize(max(0, p~ - q~)) over the anchor's support (warp 0).  q~: the first nq entries of
// sh.list_* with log-normaliser lse_q (softmax q), or the point mass at the rejected token.
__device__ void draw_residual(const TopkParams& P, const TopkShared& sh, const int* s_n, const double* s_lse, int b, int rej,
                              int a, int nq, double lse_q, uint32_t step) {
  const int lane = threadIdx.x & 31;
  if (threadIdx.x >= 32) return;
  const double inv_t = (double)P.inv_t;
  const int x = P.block_tok[(size_t)b * P.Q + rej];
  const int r = rej - 1, n = s_n[r];
  const float* v = P.list_val + ((size_t)b * P.Q + r) * kMaxTopK;
  const int* ix = P.list_idx + ((size_t)b * P.Q + r) * kMaxTopK;
  const uint32_t tagpos = (ISD_TAG_FINAL << 16) | (uint32_t)rej;
  double best = -INFINITY, best_p = -INFINITY;
  int tok = -1, tok_p = -1;  // residual draw; draw from p~ with the same noise (fallback for an empty residual)
  for (int i = lane; i < n; i += 32) {
    const double lp = (double)ldcg_f(v + i) * inv_t;
    if (isinf(lp) && lp < 0) continue;
    const int id = ldcg_i(ix + i);
    const double g = gumbel_at(P, step, b, tagpos, id);
    const double pi = exp(lp - s_lse[r]);
    double qi = 0.0;
    if (P.q_mode == 0) {
      for (int t = 0; t < nq; ++t)
        if (sh.list_idx[t] == id) qi = exp((double)sh.list_val[t] * inv_t - lse_q);
    } else {
      qi = (id == x) ? 1.0 : 0.0;
    }
    const double rr = pi - qi;
    if (rr > 0.0) {
      const double sc = log(rr) + g;
      if (tok < 0 || sc > best || (sc == best && id < tok)) { best = sc; tok = id; }
    }
    const double scp = lp - s_lse[r] + g;
    if (tok_p < 0 || scp > best_p || (scp == best_p && id < tok_p)) { best_p = scp; tok_p = id; }
  }
  warp_argmax(best, tok);
  warp_argmax(best_p, tok_p);
  if (lane == 0) {
    if (tok < 0) {
      tok = tok_p;
      atomicOr(&P.slot_status[b], ISD_ST_EMPTY_RESIDUAL);
      atomicOr(P.global_status, ISD_ST_EMPTY_RESIDUAL);
    }
    P.out.repl_tok[b] = tok;
    P.out.out_tok[(size_t)b * P.N + a] = tok;
  }
}

// ------------------------------------------------------------------------------------------------
// Pass 1: the top-k list of every valid row
// ------------------------------------------------------------------------------------------------
template <int DT>
__device__ __forceinline__ void topk_rows_body(const TopkParams& P, TopkShared& sh) {
  const int b = blockIdx.x, r = blockIdx.y;
  if (!P.active[b]) return;
  const int nv = P.n_ver[b];
  if (nv < 0 || nv > P.N - 1) {
    if (r == 0 && threadIdx.x == 0) {
      atomicOr(&P.slot_status[b], ISD_ST_SLOT_CAPACITY);
      atomicOr(P.global_status, ISD_ST_SLOT_CAPACITY);
    }
    return;
  }
  if (r >= nv + P.N) return;
  const size_t elt = DT == ISD_LOGITS_BF16 ? 2 : 4;
  const char* row = reinterpret_cast<const char*>(P.logits_cur) + ((size_t)b * P.Q + r) * (size_t)P.V * elt;
  if (!block_topk<DT>(sh, row, 0, P.V, P.top_k, P.wait_ns) && threadIdx.x == 0) {
    atomicOr(&P.slot_status[b], ISD_ST_KERNEL_TIMEOUT);
    atomicOr(P.global_status, ISD_ST_KERNEL_TIMEOUT);
  }
  const size_t base = ((size_t)b * P.Q + r) * kMaxTopK;
  if (threadIdx.x < sh.list_n) {
    P.list_val[base + threadIdx.x] = sh.list_val[threadIdx.x];
    P.list_idx[base + threadIdx.x] = sh.list_idx[threadIdx.x];
  }
  if (threadIdx.x == 0) P.list_n[(size_t)b * P.Q + r] = sh.bad ? -1 - sh.list_n : sh.list_n;
  // ---- the CTA that finishes the slot's last row runs the slot's accept phase (nobody waits for anybody)
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const int done = atomicAdd(&P.row_ticket[b], 1);
    sh.have = done == nv + P.N - 1;
    if (sh.have) P.row_ticket[b] = 0;  // ready for the next launch
  }
  __syncthreads();
  if (!sh.have) return;
  __threadfence();
  SlotScratch& S = *reinterpret_cast<SlotScratch*>(sh.ring.stage);
  slot_accept(P, S, b, nv);
  // ---- and the slot's draws, unless the proposal-law row of a rejection has to be streamed (decide kernel)
  const uint32_t step = P.step_dev ? *P.step_dev : P.step;
  const int a = S.a, rej = S.rej;
  draw_proposals(P, S.n, S.lse, b, nv, step, a >= 0 && rej == 0);
  if (a < 0) return;  // frozen: no emission
  if (rej == 0) {
    draw_bonus(P, S.n, b, nv, a, step);
  } else if (P.q_mode != 0) {
    draw_residual(P, sh, S.n, S.lse, b, rej, a, 0, 0.0, step);
  } else if (P.q_prev != nullptr && P.prev_valid) {
    // the row was a [MASK] row of the previous call, which selected its top-k already: no second stream
    const int q_row = P.q_row0[b] + rej - 1;
    const size_t pbase = ((size_t)b * P.Q + q_row) * kMaxTopK;
    int pn = P.prev_n[(size_t)b * P.Q + q_row];
    if (pn < 0) pn = -1 - pn;
    if (threadIdx.x < pn) {
      sh.list_val[threadIdx.x] = P.prev_val[pbase + threadIdx.x];
      sh.list_idx[threadIdx.x] = P.prev_idx[pbase + threadIdx.x];
    }
    __syncthreads();
    if (threadIdx.x < 32) {
      double lse_q;
      const int nq = warp_nucleus<false>(sh.list_val, pn, (double)P.inv_t, (double)P.top_p, S.w[0], lse_q);
      draw_residual(P, sh, S.n, S.lse, b, rej, a, nq, lse_q, step);
    }
  }
}

template <int DT>
__global__ void __launch_bounds__(kThreads + 32, 5) topk_rows_kernel(const TopkParams P) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  TopkShared& sh = *reinterpret_cast<TopkShared*>(smem_raw);
  // Inside isd_step the kernel ahead of this one is the attention's combine kernel, of which the selection and
  // the draws need nothing (the step's logits and the slots' state were complete before the step's first kernel
  // returned from its own wait): the pass starts at once and waits before it ends - before the commit rewrites the
  // state the attention read - which keeps the order of completion along the chain.
  if (!P.rows_early) pdl_wait();
  pdl_launch_dependents();
  topk_rows_body<DT>(P, sh);
  if (P.rows_early) pdl_wait();
  if (!P.fuse_commit) return;
  // ---- isd_step, when this kernel is the whole verification: the CTA that finishes last (a ticket over the grid;
  // nobody waits) commits the batch
  __shared__ int sm_commit[36];
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const int arrived = atomicAdd(P.step_ticket, 1);
    sm_commit[35] = (arrived == (int)(gridDim.x * gridDim.y) - 1);
  }
  __syncthreads();
  if (!sm_commit[35]) return;
  if (threadIdx.x == 0) *P.step_ticket = 0;  // ready for the next call
  __threadfence();
  commit_block(P.commit, sm_commit, sm_commit + 33);
}

// ------------------------------------------------------------------------------------------------
// Pass 2: everything else, one CTA per slot
// ------------------------------------------------------------------------------------------------
template <int DT>
__global__ void __cluster_dims__(kQSplit, 1, 1) __launch_bounds__(kThreads + 32) topk_decide_kernel(const TopkParams P) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  TopkShared& sh = *reinterpret_cast<TopkShared*>(smem_raw);
  __shared__ int s_n[32];
  __shared__ double s_lse[32];
  __shared__ double s_w[kMaxTopK];
  // Launched only when rejections need a proposal-law row that no list of the previous call covers (softmax q,
  // q_prev given, not the previous call's buffer).  A cluster of kQSplit CTAs per slot: each selects the top-k of
  // one piece of the row, the first one merges the pieces and draws the replacement.  All CTAs of a cluster read
  // the same decision, so they leave before the cluster barrier together or not at all.
  const int b = blockIdx.x / kQSplit, piece = blockIdx.x % kQSplit;
  const bool lead = piece == 0;
  pdl_wait();
  pdl_launch_dependents();
  if (!P.active[b]) return;
  const int nv = P.n_ver[b];
  if (nv < 0 || nv > P.N - 1) return;
  const int a = P.q_dec[2 * b], rej = P.q_dec[2 * b + 1];
  if (a < 0 || rej == 0) return;
  const int q_len = nv + P.N;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t step = P.step_dev ? *P.step_dev : P.step;
  const size_t elt = DT == ISD_LOGITS_BF16 ? 2 : 4;
  if (lead && threadIdx.x < q_len) {
    s_n[threadIdx.x] = P.nuc_n[(size_t)b * P.Q + threadIdx.x];
    s_lse[threadIdx.x] = P.nuc_lse[(size_t)b * P.Q + threadIdx.x];
  }
  const int q_row = P.q_row0[b] + rej - 1;
  const char* qrow = reinterpret_cast<const char*>(P.q_prev) + ((size_t)b * P.Q + q_row) * (size_t)P.V * elt;
  // every CTA of the cluster selects the top-k of its piece of the row (whole stages); their union holds the row's
  const int stage_elems = kRowStageBytes / (int)elt;
  const int per = ((P.V + stage_elems - 1) / stage_elems + kQSplit - 1) / kQSplit * stage_elems;
  const int e_lo = piece * per < P.V ? piece * per : P.V;
  const int e_hi = e_lo + per < P.V ? e_lo + per : P.V;
  if (!block_topk<DT>(sh, qrow, e_lo, e_hi, P.top_k, P.wait_ns) && threadIdx.x == 0) {
    atomicOr(&P.slot_status[b], ISD_ST_KERNEL_TIMEOUT);
    atomicOr(P.global_status, ISD_ST_KERNEL_TIMEOUT);
  }
  if (threadIdx.x < sh.list_n)
    P.q_key[((size_t)b * kQSplit + piece) * kMaxTopK + threadIdx.x] = cand_key(sh.list_val[threadIdx.x], sh.list_idx[threadIdx.x]);
  if (threadIdx.x == 0) P.q_n[(size_t)b * kQSplit + piece] = sh.list_n;
  __threadfence();
  cooperative_groups::this_cluster().sync();
  if (!lead) return;
  if (threadIdx.x < kThreads) {
    int total = 0;
    for (int r = 0; r < kQSplit; ++r) {
      const int n_r = P.q_n[(size_t)b * kQSplit + r];
      if (threadIdx.x < n_r) sh.key[total + threadIdx.x] = P.q_key[((size_t)b * kQSplit + r) * kMaxTopK + threadIdx.x];
      total += n_r;
    }
    worker_sync();
    const int n = rank_select(sh.key, total, P.top_k, sh.sorted);  // total <= kQSplit * kMaxTopK = kThreads
    if (threadIdx.x < n) {
      sh.list_val[threadIdx.x] = key_value(sh.sorted[threadIdx.x]);
      sh.list_idx[threadIdx.x] = key_index(sh.sorted[threadIdx.x]);
    }
    if (threadIdx.x == 0) sh.list_n = n;
  }
  __syncthreads();
  if (warp == 0) {
    double lse_q;
    const int nq = warp_nucleus<false>(sh.list_val, sh.list_n, (double)P.inv_t, (double)P.top_p, s_w, lse_q);
    draw_residual(P, sh, s_n, s_lse, b, rej, a, nq, lse_q, step);
  }
  (void)lane;
}

constexpr size_t kTopkSmem = sizeof(TopkShared);
static_assert(kQSplit * kMaxTopK <= kThreads, "the merge of the piece lists ranks one key per thread");

}  // namespace

int isd_verify_topk_create(isd_ctx* ctx) {
  const isd_config& c = ctx->cfg;
  const size_t rows = (size_t)c.batch * ctx->Q;
  // two sets of lists: this call's and the previous call's
  if (cudaMalloc(&ctx->topk_val, 2 * sizeof(float) * rows * kMaxTopK) != cudaSuccess) return ISD_ERR_NO_MEMORY;
  if (cudaMalloc(&ctx->topk_idx, 2 * sizeof(int) * rows * kMaxTopK) != cudaSuccess) return ISD_ERR_NO_MEMORY;
  if (cudaMalloc(&ctx->topk_n, 2 * sizeof(int) * rows) != cudaSuccess) return ISD_ERR_NO_MEMORY;
  cudaMemset(ctx->topk_n, 0, 2 * sizeof(int) * rows);
  ctx->topk_cur = 0;
  ctx->topk_prev_rows = nullptr;
  if (cudaMalloc(&ctx->topk_q_key, sizeof(unsigned long long) * (size_t)c.batch * kQSplit * kMaxTopK) != cudaSuccess) return ISD_ERR_NO_MEMORY;
  // ints: piece counts [B, kQSplit], decisions [B, 2], supports and flags [B, Q] each, row tickets [B]
  const size_t n_ints = (size_t)c.batch * (kQSplit + 2 + 2 * ctx->Q + 1);
  if (cudaMalloc(&ctx->topk_q_n, sizeof(int) * n_ints) != cudaSuccess) return ISD_ERR_NO_MEMORY;
  cudaMemset(ctx->topk_q_n, 0, sizeof(int) * n_ints);
  if (cudaMalloc(&ctx->topk_nuc_lse, sizeof(double) * rows) != cudaSuccess) return ISD_ERR_NO_MEMORY;
  cudaError_t e = cudaSuccess;
  if (e == cudaSuccess) e = cudaFuncSetAttribute(topk_rows_kernel<ISD_LOGITS_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTopkSmem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(topk_rows_kernel<ISD_LOGITS_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTopkSmem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(topk_decide_kernel<ISD_LOGITS_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTopkSmem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(topk_decide_kernel<ISD_LOGITS_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTopkSmem);
  return e == cudaSuccess ? ISD_OK : ISD_ERR_CUDA;
}

void isd_verify_topk_destroy(isd_ctx* ctx) {
  cudaFree(ctx->topk_val);
  cudaFree(ctx->topk_idx);
  cudaFree(ctx->topk_n);
  cudaFree(ctx->topk_q_key);
  cudaFree(ctx->topk_q_n);
  cudaFree(ctx->topk_nuc_lse);
  ctx->topk_val = nullptr;
  ctx->topk_idx = nullptr;
  ctx->topk_n = nullptr;
  ctx->topk_q_key = nullptr;
  ctx->topk_q_n = nullptr;
  ctx->topk_nuc_lse = nullptr;
}

int isd_launch_verify_topk(isd_ctx* ctx, const isd_batch_state* st, const void* logits_cur,
                           const void* q_prev_logits, uint32_t step, const isd_verify_out* out,
                           cudaStream_t stream, isd_batch_state* commit_st, bool* committed) {
  const isd_config& c = ctx->cfg;
  TopkParams P;
  P.B = c.batch; P.N = c.stride; P.Q = ctx->Q; P.V = c.vocab;
  P.logits_dtype = c.logits_dtype; P.q_mode = c.q_mode; P.propose_mode = c.propose_mode; P.top_k = c.top_k;
  P.inv_t = c.inv_temperature; P.tau = c.tau; P.top_p = c.top_p;
  P.wait_ns = ctx->wait_ns;
  P.seed_lo = (uint32_t)c.seed; P.seed_hi = (uint32_t)(c.seed >> 32); P.step = step;
  P.step_dev = ctx->step_counter;
  P.n_ver = st->n_ver; P.active = st->active; P.block_tok = st->block_tok; P.q_row0 = st->q_row0;
  P.q_stats = st->q_stats; P.slot_status = st->slot_status; P.global_status = ctx->global_status;
  P.logits_cur = logits_cur; P.q_prev = q_prev_logits; P.out = *out;
  const size_t rows = (size_t)c.batch * ctx->Q;
  const int cur = ctx->topk_cur, prv = cur ^ 1;
  P.list_val = ctx->topk_val + cur * rows * kMaxTopK; P.list_idx = ctx->topk_idx + cur * rows * kMaxTopK;
  P.list_n = ctx->topk_n + cur * rows;
  P.prev_val = ctx->topk_val + prv * rows * kMaxTopK; P.prev_idx = ctx->topk_idx + prv * rows * kMaxTopK;
  P.prev_n = ctx->topk_n + prv * rows;
  // the proposal-law rows are the [MASK] rows of the previous step's logits: when that buffer is the one the previous
  // call selected from, its lists are reused instead of streaming the rows again
  // (and when this call is the step right after it; with a device-resident step number the host cannot tell)
  P.prev_valid = (q_prev_logits != nullptr && q_prev_logits == ctx->topk_prev_rows && ctx->step_counter == nullptr &&
                  step == ctx->topk_prev_step + 1u) ? 1 : 0;
  ctx->topk_cur = prv;
  ctx->topk_prev_rows = logits_cur;
  ctx->topk_prev_step = step;
  P.q_key = ctx->topk_q_key; P.q_n = ctx->topk_q_n; P.q_dec = ctx->topk_q_n + (size_t)c.batch * kQSplit;
  P.nuc_n = P.q_dec + 2 * (size_t)c.batch; P.nuc_bad = P.nuc_n + (size_t)c.batch * ctx->Q;
  P.row_ticket = P.nuc_bad + (size_t)c.batch * ctx->Q; P.nuc_lse = ctx->topk_nuc_lse;
  const dim3 grid1(c.batch, ctx->Q);
  // a second kernel only when rejections need proposal-law rows that have to be streamed
  const bool stream_q = c.q_mode == 0 && q_prev_logits != nullptr && !P.prev_valid;
  // the row kernel commits by itself when it is the whole verification (no decide kernel after it)
  P.fuse_commit = (commit_st != nullptr && !stream_q && ctx->step_ticket != nullptr) ? 1 : 0;
  P.rows_early = commit_st != nullptr;  // called from isd_step / isd_step_layers, behind the step's attention
  P.step_ticket = ctx->step_ticket;
  P.commit = make_commit_params(ctx, P.fuse_commit ? commit_st : st, out);
  if (committed) *committed = P.fuse_commit != 0;
  if (ctx->ev_verify0) cudaEventRecord(ctx->ev_verify0, stream);
  cudaError_t e;
  if (c.logits_dtype == ISD_LOGITS_BF16) {
    e = isd_launch_pdl(topk_rows_kernel<ISD_LOGITS_BF16>, grid1, dim3(kThreads + 32), kTopkSmem, stream, P);
    if (stream_q) topk_decide_kernel<ISD_LOGITS_BF16><<<c.batch * kQSplit, kThreads + 32, kTopkSmem, stream>>>(P);
  } else {
    e = isd_launch_pdl(topk_rows_kernel<ISD_LOGITS_F32>, grid1, dim3(kThreads + 32), kTopkSmem, stream, P);
    if (stream_q) topk_decide_kernel<ISD_LOGITS_F32><<<c.batch * kQSplit, kThreads + 32, kTopkSmem, stream>>>(P);
  }
  if (ctx->ev_verify1) cudaEventRecord(ctx->ev_verify1, stream);
  ctx->launches += stream_q ? 2 : 1;
  return (e == cudaSuccess && cudaGetLastError() == cudaSuccess) ? ISD_OK : ISD_ERR_CUDA;
}
