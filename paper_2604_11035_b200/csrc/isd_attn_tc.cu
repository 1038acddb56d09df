// isd_attn tensor-core path (sm_100a): strict-causal attention of every slot's ISD query block
// against its paged bf16 KV cache (Sec. 3.1 mask; Sec. 3.3 (1) "single paged-only kernel" for the
// 2N-1 row extend), re-designed for B200:
//
//   * GQA packing: the G = Hq/Hkv query heads that share a KV head and the q_len block rows form one
//     M = 128 row tile (row m = r * G + head-in-group), so each KV byte is read once per step.
//   * KV pages (16 tokens x 128 dims, 4 KiB per head) are staged by TMA (cp.async.bulk.tensor, every
//     CTA loads for itself) into a 6-deep shared-memory ring in the 128-byte-swizzled layout tcgen05 consumes;
//     one 128-key tile = 8 pages.
//   * S = Q K^T and O += P V run on the 5th-gen tensor cores (tcgen05.mma, cta_group::1, M=128,
//     N=128, K=16, bf16 -> fp32) with accumulators in TMEM; S is double-buffered so that the
//     softmax of tile j overlaps the QK^T of tile j+1.  Both A operands live in TMEM (Q for QK^T,
//     P -- written over its own S tile -- for PV), so shared memory holds nothing but the KV ring and
//     each MMA fetches only its 4 KiB B operand from it.
//   * Softmax: 128 threads, one TMEM lane (= row) each, so row max / sum need no shuffles; the
//     running maximum is only raised when it grows by more than 2^8 (lazy rescale of O in TMEM).
//   * Persistent CTAs, one per SM.  All (slot, kv-head) KV ranges are laid end to end in units of
//     128-key tiles and cut into equal contiguous shares, so every CTA streams the same number of
//     bytes; a share's ragged first/last pieces go to a small fp32 scratch and are merged by a
//     second kernel (log-sum-exp combine).  Nothing waits on another CTA.
//   * Warp roles: warps 0-3 softmax/epilogue, warps 4-6 TMA producers (round-robin over the ring
//     stages: issuing the 16 copies of a stage costs one warp about a microsecond), warp 7 MMA issuer.
//
// Every mbarrier wait is bounded; on expiry the CTA raises ISD_ST_KERNEL_TIMEOUT in the global status
// word, stops issuing work, drains, frees its TMEM and returns.
#include <cuda.h>
#include <new>

#include "isd_internal.cuh"

namespace {

constexpr int kTile = 128;                 // keys per tile
constexpr int kStageBytes = 32768;         // one K or V tile: [half(2)][page(8)][tok(16)][128 B]
constexpr int kStages = 6;
constexpr int kSegCost = 4;  // fixed cost of a segment in units of one tile's time (split axis), measured
constexpr int kThreads = 256;
constexpr int kProducerWarps = 3;        // warps 4..6 issue the TMA copies round-robin, warp 7 issues the MMAs
constexpr int kSmRing = 0;
constexpr int kSmBar = kSmRing + kStages * kStageBytes;  // 196608
constexpr int kSmMl = kSmBar + 256;     // [128][2] floats: (max, sum) of every replica row at segment end
constexpr int kSmXchg = kSmMl + 1024;   // [3][32 rows] or [1][64 rows] x 32 floats: rows handed to replica 0
// TMEM columns (512 allocated): S double buffer (P, as bf16 pairs, overwrites the first 64 columns of
// its S buffer once the scores are in registers), O, and the query block Q (bf16 pairs, 64 columns)
constexpr uint32_t kTmS = 0, kTmO = 256, kTmQ = 384;  // Q: two buffers of 64 columns (segment parity)
constexpr int kSmPrefix = kSmXchg + 12288;  // tile prefix over slots when the batch fits (else it stays in global memory)
constexpr int kMaxSmemPrefixSlots = 1024;
constexpr int kSmSlot = kSmPrefix + (kMaxSmemPrefixSlots + 1) * 4 + 12;  // per slot: ctx_len | q_len << 24 (with the prefix)
constexpr int kSmemBytes = kSmSlot + kMaxSmemPrefixSlots * 4;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// barrier slots (8 bytes each) inside the barrier block
enum { BAR_FULL = 0, BAR_EMPTY = kStages, BAR_SFULL = 2 * kStages,
       BAR_PFULL = 2 * kStages + 2, BAR_ODONE = 2 * kStages + 4, BAR_OFREE = 2 * kStages + 6,
       BAR_QFULL = 2 * kStages + 7, BAR_COUNT = 2 * kStages + 8 };

struct TcParams {
  int B, Q, N, Hq, Hkv, G, max_pages, num_pages;
  float scale2;  // sm_scale * log2(e)
  const int32_t* ctx_len;
  const int32_t* n_ver;
  const uint8_t* active;
  const int32_t* page_table;
  const uint32_t* slot_status;
  uint32_t* global_status;
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  float* lse;
  int* tile_prefix;  // [B + 1] split-axis length (tiles + kSegCost) per kv head, exclusive prefix over slots
  float* part_o;     // [ctas * 2][128][128]
  float* part_ml;    // [ctas * 2][128][2]
  int num_ctas;
  unsigned long long wait_ns;  // time limit of a device-side wait
};

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}

// Bounded wait: returns false (and raises the abort flag) when the time limit is reached or another thread of
// the CTA has given up.  The limit (nanoseconds) sits in shared memory two words behind the abort flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long budget = *reinterpret_cast<const volatile unsigned long long*>(abort_flag + 2);
  return isd_bounded_wait(budget, abort_flag, [&]() { return mbar_try_wait(bar, parity); });
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}

// One lane of a converged warp; unlike `lane == 0` the compiler keeps the surrounding code uniform, so
// that MMA descriptors stay in uniform registers instead of being moved there one by one.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred = 0;
  asm volatile(
      "{\n.reg .b32 rx;\n.reg .pred px;\n"
      "elect.sync rx|px, 0xffffffff;\n"
      "selp.u32 %0, 1, 0, px;\n}"
      : "=r"(pred));
  return pred != 0;
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// A operand read from tensor memory (row = lane, 2 bf16 per 32-bit column), B from shared memory
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accum) : "memory");
}


// K-major / MN-major shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  const uint32_t lo = ((addr & 0x3FFFFu) >> 4) | ((lbo_bytes >> 4) << 16);
  const uint32_t hi = (sbo_bytes >> 4) | (1u << 14) | (2u << 29);
  return ((uint64_t)hi << 32) | lo;
}

#define TMEM_LD32(taddr, v, o)                                                                          \
  asm volatile(                                                                                         \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                         \
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25," \
      "%26,%27,%28,%29,%30,%31}, [%32];"                                                                \
      : "=r"(v[o + 0]), "=r"(v[o + 1]), "=r"(v[o + 2]), "=r"(v[o + 3]), "=r"(v[o + 4]), "=r"(v[o + 5]), \
        "=r"(v[o + 6]), "=r"(v[o + 7]), "=r"(v[o + 8]), "=r"(v[o + 9]), "=r"(v[o + 10]),                \
        "=r"(v[o + 11]), "=r"(v[o + 12]), "=r"(v[o + 13]), "=r"(v[o + 14]), "=r"(v[o + 15]),            \
        "=r"(v[o + 16]), "=r"(v[o + 17]), "=r"(v[o + 18]), "=r"(v[o + 19]), "=r"(v[o + 20]),            \
        "=r"(v[o + 21]), "=r"(v[o + 22]), "=r"(v[o + 23]), "=r"(v[o + 24]), "=r"(v[o + 25]),            \
        "=r"(v[o + 26]), "=r"(v[o + 27]), "=r"(v[o + 28]), "=r"(v[o + 29]), "=r"(v[o + 30]),            \
        "=r"(v[o + 31])                                                                                 \
      : "r"(taddr))

#define TMEM_ST32(taddr, v, o)                                                                          \
  asm volatile(                                                                                         \
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "                                                   \
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26," \
      "%27,%28,%29,%30,%31,%32};"                                                                       \
      ::"r"(taddr), "r"(v[o + 0]), "r"(v[o + 1]), "r"(v[o + 2]), "r"(v[o + 3]), "r"(v[o + 4]),          \
        "r"(v[o + 5]), "r"(v[o + 6]), "r"(v[o + 7]), "r"(v[o + 8]), "r"(v[o + 9]), "r"(v[o + 10]),      \
        "r"(v[o + 11]), "r"(v[o + 12]), "r"(v[o + 13]), "r"(v[o + 14]), "r"(v[o + 15]), "r"(v[o + 16]), \
        "r"(v[o + 17]), "r"(v[o + 18]), "r"(v[o + 19]), "r"(v[o + 20]), "r"(v[o + 21]), "r"(v[o + 22]), \
        "r"(v[o + 23]), "r"(v[o + 24]), "r"(v[o + 25]), "r"(v[o + 26]), "r"(v[o + 27]), "r"(v[o + 28]), \
        "r"(v[o + 29]), "r"(v[o + 30]), "r"(v[o + 31])                                                  \
      : "memory")

#define TMEM_ST16(taddr, v, o)                                                                          \
  asm volatile(                                                                                         \
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "                                                   \
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"                                       \
      ::"r"(taddr), "r"(v[o + 0]), "r"(v[o + 1]), "r"(v[o + 2]), "r"(v[o + 3]), "r"(v[o + 4]),          \
        "r"(v[o + 5]), "r"(v[o + 6]), "r"(v[o + 7]), "r"(v[o + 8]), "r"(v[o + 9]), "r"(v[o + 10]),      \
        "r"(v[o + 11]), "r"(v[o + 12]), "r"(v[o + 13]), "r"(v[o + 14]), "r"(v[o + 15])                  \
      : "memory")

__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

// bf16 pair (a in the low half, b in the high half) with the conversion instruction: one instruction instead of
// three, which matters more than the pipe it runs on -- the softmax warps are bound by instruction issue (one warp
// per scheduler), not by the transcendental unit
__device__ __forceinline__ uint32_t pack_bf16_cvt(float a, float b) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(b), "f"(a));
  return d;
}

// ------------------------------------------------------------------------------------------------
// Work split: identical, independent enumeration in every warp role
// ------------------------------------------------------------------------------------------------
struct Segment {
  int b, g;      // slot, kv head
  int j0, j1;    // tiles [j0, j1) of the pair
  int T;         // tiles of the whole pair
  int kv_len;    // ctx_len + q_len
  int ctx, q_len;
  int part_slot; // scratch slot when the segment does not cover the whole pair, else -1
};

// Units of the split axis per CTA.  Small batches do not fill the machine: below kMinShare units a share would
// be mostly fixed cost (Q staging, pipeline fill, a partial result of 64 KB that the combine kernel reads back), so
// fewer CTAs take longer shares and the rest leave at once.
constexpr int kMinShare = 8;  // 12 and 16 measured slower at batch 1, equal at batch 8
__device__ __forceinline__ long long share_units(long long total, int num_ctas) {
  const long long per = (total + num_ctas - 1) / num_ctas;
  return per < kMinShare ? kMinShare : per;
}

struct WorkIter {
  const int* prefix;
  const int* slot_info;  // ctx_len | q_len << 24 per slot in shared memory, or nullptr (read the state arrays)
  int B, Hkv, b;
  long long t, t_begin, t_end;
  __device__ void init(const TcParams& P, int cta, const int* prefix_, const int* slot_info_) {
    prefix = prefix_;
    slot_info = slot_info_;
    B = P.B; Hkv = P.Hkv;
    const long long total = (long long)prefix[B] * Hkv;
    const long long per = share_units(total, P.num_ctas);
    t_begin = t = (long long)cta * per;
    t_end = t + per < total ? t + per : total;
    // first slot whose range ends after t
    int lo = 0, hi = B;
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if ((long long)prefix[mid + 1] * Hkv > t) hi = mid; else lo = mid + 1;
    }
    b = lo;
  }
  __device__ bool next(const TcParams& P, int cta, Segment& s) {
    for (;;) {
      if (t >= t_end) return false;
      while (b < B && (long long)prefix[b + 1] * Hkv <= t) ++b;
      if (b >= B) return false;
      // positions of a pair on the split axis: kSegCost units of fixed cost, then its tiles
      const int Tv = prefix[b + 1] - prefix[b];
      const long long off = t - (long long)prefix[b] * Hkv;
      const int v0 = (int)(off % Tv);
      const long long room = t_end - t;
      const int v1 = (long long)(Tv - v0) <= room ? Tv : v0 + (int)room;
      const bool first = (t == t_begin);
      t += v1 - v0;
      const int T = Tv - kSegCost;
      s.j0 = v0 > kSegCost ? v0 - kSegCost : 0;
      s.j1 = v1 > kSegCost ? v1 - kSegCost : 0;
      if (s.j1 <= s.j0) continue;  // only (part of) the fixed-cost units of the pair fell into this share
      s.b = b; s.T = T;
      s.g = (int)(off / Tv);
      if (slot_info) {
        const int w = slot_info[b];
        s.ctx = w & 0xFFFFFF;
        s.q_len = (int)((unsigned)w >> 24);
      } else {
        s.ctx = P.ctx_len[b];
        s.q_len = P.n_ver[b] + P.N;
      }
      s.kv_len = s.ctx + s.q_len;
      const bool whole = (s.j0 == 0 && s.j1 == T);
      s.part_slot = whole ? -1 : cta * 2 + (first ? 0 : 1);
      return true;
    }
  }
};

// Length of a slot's (slot, kv head) pairs on the split axis: its 128-key tiles plus kSegCost units for the
// fixed cost of a segment (Q staging, pipeline fill and drain, epilogue: measured at about the time of four
// tiles).  Shares of equal length on this axis take equal time whether they hold a few long pairs or many
// short ones; with tiles alone the CTAs with the most segments finished 10 % after the average.
__device__ __forceinline__ int slot_tiles(const TcParams& P, int b) {
  if (b >= P.B || !P.active[b]) return 0;
  const int nv = P.n_ver[b];
  const int ctx = P.ctx_len[b];
  const bool ok = nv >= 0 && nv <= P.N - 1 && ctx >= 0 &&
                  (P.slot_status[b] & (ISD_ST_BAD_PAGE_ID | ISD_ST_SLOT_CAPACITY)) == 0;
  return ok ? (ctx + nv + P.N + kTile - 1) / kTile + kSegCost : 0;
}

// Exclusive prefix of tiles per slot, computed by the 256 threads of a main-kernel CTA into shared
// memory (batches up to kMaxSmemPrefixSlots); CTA 0 also publishes it for the combine kernel.
__device__ void block_tile_prefix(const TcParams& P, int* sm_prefix, int* sm_slot, int* sm_warp, bool publish) {
  int carry = 0;
  for (int base = 0; base < P.B; base += kThreads) {
    const int b = base + threadIdx.x;
    const int tiles = slot_tiles(P, b);
    if (b < P.B && tiles > 0) sm_slot[b] = (P.ctx_len[b] & 0xFFFFFF) | ((P.n_ver[b] + P.N) << 24);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = tiles;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += v;
    }
    if (lane == 31) sm_warp[warp] = inc;
    __syncthreads();
    int woff = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) {
      const int x = sm_warp[w];
      if (w < warp) woff += x;
      tot += x;
    }
    if (b < P.B) {
      const int excl = carry + woff + inc - tiles;
      sm_prefix[b] = excl;
      if (publish) P.tile_prefix[b] = excl;
    }
    carry += tot;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    sm_prefix[P.B] = carry;
    if (publish) P.tile_prefix[P.B] = carry;
  }
  __syncthreads();
}

// ------------------------------------------------------------------------------------------------
// Plan for batches too large for the in-kernel prefix: tiles per slot and their exclusive prefix
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) attn_plan_kernel(const TcParams P) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ int sm_warp[33];
  __shared__ int sm_carry;
  if (threadIdx.x == 0) sm_carry = 0;
  __syncthreads();
  for (int base = 0; base < P.B; base += 1024) {
    const int b = base + threadIdx.x;
    const int tiles = slot_tiles(P, b);
    // inclusive scan
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = tiles;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += v;
    }
    if (lane == 31) sm_warp[warp] = inc;
    __syncthreads();
    if (warp == 0) {
      int w = sm_warp[lane], winc = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += v;
      }
      sm_warp[lane] = winc - w;
      if (lane == 31) sm_warp[32] = winc;
    }
    __syncthreads();
    const int excl = sm_carry + sm_warp[warp] + inc - tiles;
    if (b < P.B) P.tile_prefix[b] = excl;
    __syncthreads();
    if (threadIdx.x == 0) sm_carry += sm_warp[32];
    __syncthreads();
  }
  if (threadIdx.x == 0) P.tile_prefix[P.B] = sm_carry;
}

// ------------------------------------------------------------------------------------------------
// Softmax / epilogue of one segment, executed by the 128 threads of warps 0-3 (thread = TMEM lane).
//
// Key split across lane groups: when a block has at most 128 / F valid rows (F = 2 or 4) the query
// rows are replicated F times along M, and replica `part` only keeps the keys
// [part * 128 / F, (part + 1) * 128 / F) of every tile (the others get probability 0).  Each thread then
// evaluates 128 / F exponentials per tile instead of 128 -- the transcendental unit is the busiest pipe
// of this kernel -- and all four schedulers share the valid rows.  The replicas are independent
// online-softmax streams with their own running maximum; they are merged (log-sum-exp) once per
// segment through a small shared-memory buffer, or by the combine kernel for split segments.
// ------------------------------------------------------------------------------------------------
struct SoftmaxCtx {
  uint8_t* smem;
  uint32_t bar_base;
  volatile int* abort_flag;
  uint32_t tmem_s0, tmem_o, tmem_q;
  uint32_t n, seg;
};

__device__ __forceinline__ void softmax_group_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Replication factor of a segment's rows along M (see softmax_segment)
__device__ __forceinline__ int seg_replicas(const TcParams& P, const Segment& sg) {
  const int rows_valid = sg.q_len * P.G;
  return rows_valid > 64 ? 1 : (rows_valid > 32 ? 2 : 4);
}

__device__ __forceinline__ const __nv_bfloat16* q_row_ptr(const TcParams& P, const Segment& sg, int m, bool& row_ok) {
  const int RG = 128 / seg_replicas(P, sg);
  const int v = m % RG;
  const int r = v / P.G, hg = v % P.G;
  row_ok = v < sg.q_len * P.G;
  return P.q + (((size_t)sg.b * P.Q + (row_ok ? r : 0)) * P.Hq + sg.g * P.G + hg) * ISD_HEAD_DIM;
}

// Stage the query block of a segment (logical row v = r * G + head-in-group, 128 bf16 = 64 packed
// columns, replicated along M, padding rows zero) into Q buffer `seg & 1` of tensor memory and announce
// it.  The buffer's previous user (segment seg - 2) finished its QK MMAs long ago.  Staging the next
// segment's block right after the current segment's last P tile lets the MMA warp issue the next QK^T
// while this segment's last PV and epilogue are still running.
__device__ __forceinline__ void stage_q(const TcParams& P, const Segment& sg, SoftmaxCtx& sc, uint32_t seg) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
  bool row_ok;
  const uint4* src = reinterpret_cast<const uint4*>(q_row_ptr(P, sg, warp * 32 + lane, row_ok));
  uint32_t qv[64];
#pragma unroll
  for (int c = 0; c < 16; ++c) {
    uint4 x = make_uint4(0, 0, 0, 0);
    if (row_ok) x = src[c];
    qv[4 * c] = x.x; qv[4 * c + 1] = x.y; qv[4 * c + 2] = x.z; qv[4 * c + 3] = x.w;
  }
  const uint32_t tq = sc.tmem_q + (seg & 1u) * 64u + lane_base;
  TMEM_ST32(tq, qv, 0);
  TMEM_ST32(tq + 32, qv, 32);
  tmem_wait_st();
  tc_fence_before();
  __syncwarp();
  if (lane == 0) mbar_arrive(sc.bar_base + 8u * (uint32_t)BAR_QFULL);
}

template <int F>
__device__ __forceinline__ bool softmax_segment(const TcParams& P, const Segment& sg, SoftmaxCtx& sc,
                                                const Segment* sg_next) {
  constexpr int RG = 128 / F;  // rows per replica group
  constexpr int C = 128 / F;   // key columns per thread and tile
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m = warp * 32 + lane;  // TMEM lane
  const int v = m % RG, part = m / RG;
  const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
  volatile int* abort_flag = sc.abort_flag;
  auto bar = [&](int i) { return sc.bar_base + 8u * (uint32_t)i; };
  const int cnt = sg.j1 - sg.j0;
  const int rows_valid = sg.q_len * P.G;
  const int r = v / P.G, hg = v % P.G;
  const bool row_ok = v < rows_valid;
  if (sg_next != nullptr) {  // pull the next segment's query rows towards L2 well before they are staged
    bool nok;
    const __nv_bfloat16* nq = q_row_ptr(P, *sg_next, m, nok);
    if (nok) {
      asm volatile("prefetch.global.L2 [%0];" ::"l"(nq));
      asm volatile("prefetch.global.L2 [%0];" ::"l"(nq + 64));
    }
  }
  float m2 = -INFINITY, l = 0.f;  // running max (log2 domain) and sum of this (row, replica)
  bool ok = true;
  for (int i = 0; i < cnt && ok; ++i) {
    const uint32_t nn = sc.n + i;
    const int j = sg.j0 + i;
    {
      ok = mbar_wait(bar(BAR_SFULL + (nn & 1u)), (nn >> 1) & 1u, abort_flag);
    }
    if (!ok) break;
    tc_fence_after();
    uint32_t sv[C];
    const uint32_t ts = sc.tmem_s0 + (nn & 1u) * 128u + lane_base;
#pragma unroll
    for (int q4 = 0; q4 < C / 32; ++q4) TMEM_LD32(ts + part * C + q4 * 32, sv, q4 * 32);
    tmem_wait_ld();
    // ---- mask (last tiles only) and row max; independent chains of 3-input max keep the single
    // softmax warp of each scheduler busy (no other warp hides the latency)
    const int kb = j * kTile + part * C;
    const int limit = row_ok ? (sg.ctx + r - kb) : -1;  // own columns c <= limit are visible
    if (limit < C - 1) {
#pragma unroll
      for (int c = 0; c < C; ++c)
        if (c > limit) sv[c] = 0xFF800000u;  // -inf
    }
    float mxa = -INFINITY, mxb = -INFINITY, mxc = -INFINITY, mxd = -INFINITY;
#pragma unroll
    for (int c = 0; c < C; c += 8) {
      mxa = max3(mxa, __uint_as_float(sv[c]), __uint_as_float(sv[c + 1]));
      mxb = max3(mxb, __uint_as_float(sv[c + 2]), __uint_as_float(sv[c + 3]));
      mxc = max3(mxc, __uint_as_float(sv[c + 4]), __uint_as_float(sv[c + 5]));
      mxd = max3(mxd, __uint_as_float(sv[c + 6]), __uint_as_float(sv[c + 7]));
    }
    const float mx = fmaxf(fmaxf(mxa, mxb), fmaxf(mxc, mxd)) * P.scale2;  // log2 domain (scale2 > 0)
    // ---- lazy rescale: raise the reference maximum only when it grows by more than 2^8
    float m_use = m2;
    const bool grow = mx > m2 + 8.f || (m2 == -INFINITY && mx > -INFINITY);
    const bool any_grow = __any_sync(0xffffffffu, grow && i > 0);
    if (grow) m_use = mx;
    if (any_grow) {
      // PV(nn-1) must have finished before O is touched.  PV completions alternate between two
      // barriers: a waiter may lag one PV behind (PV(x-2) is known complete once S(x) arrived),
      // which a single barrier's phase parity could not tell apart.
      ok = mbar_wait(bar(BAR_ODONE + ((nn - 1u) & 1u)), ((nn - 1u) >> 1) & 1u, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const float f = (grow && m2 > -INFINITY) ? ex2f(m2 - m_use) : 1.f;
      uint32_t ov[32];
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        TMEM_LD32(sc.tmem_o + lane_base + q4 * 32, ov, 0);
        tmem_wait_ld();
#pragma unroll
        for (int c = 0; c < 32; ++c) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * f);
        TMEM_ST32(sc.tmem_o + lane_base + q4 * 32, ov, 0);
      }
      tmem_wait_st();
      l *= f;
    }
    m2 = m_use;
    // ---- probabilities and row sum; P (bf16 pairs) overwrites the first 64 columns of S(nn): own
    // keys carry the probabilities, the other replicas' keys are zero
    const float mref = (m2 == -INFINITY) ? 0.f : m2;
    const uint64_t sc2 = pack2(P.scale2, P.scale2), nm2 = pack2(-mref, -mref);
    uint64_t acc[4] = {pack2(0.f, 0.f), pack2(0.f, 0.f), pack2(0.f, 0.f), pack2(0.f, 0.f)};
    // F > 1: the thread's C / 2 packed columns go straight to its replica's part of the P tile and zeros to the
    // rest (stores at run-time column offsets, no per-element selects)
    uint32_t pk[C / 2];
#pragma unroll
    for (int c = 0; c < C / 2; ++c) {
      float x0, x1;
      unpack2(fma2(pack2(__uint_as_float(sv[2 * c]), __uint_as_float(sv[2 * c + 1])), sc2, nm2), x0, x1);
      const float p0 = ex2f(x0), p1 = ex2f(x1);
      acc[c & 3] = add2(acc[c & 3], pack2(p0, p1));
      pk[c] = pack_bf16_cvt(p0, p1);
    }
    float lsum;
    {
      float a0, a1, b0, b1;
      unpack2(add2(acc[0], acc[1]), a0, a1);
      unpack2(add2(acc[2], acc[3]), b0, b1);
      lsum = (a0 + a1) + (b0 + b1);
    }
    if (F == 1) {
      TMEM_ST32(ts, pk, 0);
      TMEM_ST32(ts + 32, pk, 32);
    } else {
      uint32_t zero[32];
#pragma unroll
      for (int c = 0; c < 32; ++c) zero[c] = 0u;
      if (F == 2) {
        TMEM_ST32(ts + (uint32_t)part * 32u, pk, 0);
        TMEM_ST32(ts + (uint32_t)(1 - part) * 32u, zero, 0);
      } else {  // F = 4: own quarter, then zeros over the other quarter of the same half and over the other half
        TMEM_ST16(ts + (uint32_t)part * 16u, pk, 0);
        TMEM_ST16(ts + (uint32_t)(part ^ 1) * 16u, zero, 0);
        TMEM_ST32(ts + (uint32_t)((part >> 1) ^ 1) * 32u, zero, 0);
      }
    }
    tmem_wait_st();
    l += lsum;
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(bar(BAR_PFULL + (nn & 1u)));
  }
  if (!ok) return false;
  if (sg_next != nullptr) stage_q(P, *sg_next, sc, sc.seg + 1);
  // ---- epilogue: wait for the last PV, read O, write the result or the partial
  const uint32_t last = sc.n + cnt - 1;
  ok = mbar_wait(bar(BAR_ODONE + (last & 1u)), (last >> 1) & 1u, abort_flag);
  if (!ok) return false;
  tc_fence_after();
  if (sg.part_slot >= 0) {
    // split segment: every replica's un-normalised row goes to the scratch, the combine kernel merges
#pragma unroll
    for (int q4 = 0; q4 < 4; ++q4) {
      uint32_t ov[32];
      TMEM_LD32(sc.tmem_o + lane_base + q4 * 32, ov, 0);
      tmem_wait_ld();
      if (row_ok) {
        uint4* dst = reinterpret_cast<uint4*>(P.part_o + ((size_t)sg.part_slot * 128 + m) * 128 + q4 * 32);
#pragma unroll
        for (int c = 0; c < 8; ++c) dst[c] = make_uint4(ov[c * 4], ov[c * 4 + 1], ov[c * 4 + 2], ov[c * 4 + 3]);
      }
    }
    if (row_ok) {
      P.part_ml[((size_t)sg.part_slot * 128 + m) * 2 + 0] = m2;
      P.part_ml[((size_t)sg.part_slot * 128 + m) * 2 + 1] = l;
    }
  } else {
    // whole segment: merge the F replicas of a row (log-sum-exp), normalise, write bf16
    float* sm_ml = reinterpret_cast<float*>(sc.smem + kSmMl);
    float* sm_x = reinterpret_cast<float*>(sc.smem + kSmXchg);
    float w = (l > 0.f) ? 1.f / l : 0.f, Mrow = m2, Lrow = l;
    if (F > 1) {
      sm_ml[2 * m] = m2;
      sm_ml[2 * m + 1] = l;
      softmax_group_sync();
      Mrow = -INFINITY;
#pragma unroll
      for (int pp = 0; pp < F; ++pp) Mrow = fmaxf(Mrow, sm_ml[2 * (pp * RG + v)]);
      Lrow = 0.f;
#pragma unroll
      for (int pp = 0; pp < F; ++pp) {
        const float mp = sm_ml[2 * (pp * RG + v)], lp = sm_ml[2 * (pp * RG + v) + 1];
        Lrow += (mp == -INFINITY) ? 0.f : lp * ex2f(mp - Mrow);
      }
      w = (m2 == -INFINITY || !(Lrow > 0.f)) ? 0.f : ex2f(m2 - Mrow) / Lrow;
    }
#pragma unroll
    for (int q4 = 0; q4 < 4; ++q4) {
      uint32_t ov[32];
      TMEM_LD32(sc.tmem_o + lane_base + q4 * 32, ov, 0);
      tmem_wait_ld();
      float o[32];
#pragma unroll
      for (int c = 0; c < 32; ++c) o[c] = __uint_as_float(ov[c]) * w;
      if (F > 1) {
        // replicas 1..F-1 hand their scaled rows to replica 0 through shared memory (32 columns a round)
        // layout [replica - 1][float4 column c][row v]: consecutive threads touch consecutive 16-byte
        // words, so neither the writes nor the reads below conflict on shared-memory banks
        if (part > 0) {
          float4* dst = reinterpret_cast<float4*>(sm_x) + (size_t)(part - 1) * 8 * RG + v;
#pragma unroll
          for (int c = 0; c < 8; ++c) dst[c * RG] = make_float4(o[4 * c], o[4 * c + 1], o[4 * c + 2], o[4 * c + 3]);
        }
        softmax_group_sync();
        if (part == 0) {
#pragma unroll
          for (int pp = 1; pp < F; ++pp) {
            const float4* src = reinterpret_cast<const float4*>(sm_x) + (size_t)(pp - 1) * 8 * RG + v;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              const float4 t = src[c * RG];
              o[4 * c] += t.x; o[4 * c + 1] += t.y; o[4 * c + 2] += t.z; o[4 * c + 3] += t.w;
            }
          }
        }
        softmax_group_sync();
      }
      if (row_ok && part == 0) {
        uint4* dst = reinterpret_cast<uint4*>(
            P.out + (((size_t)sg.b * P.Q + r) * P.Hq + sg.g * P.G + hg) * ISD_HEAD_DIM + q4 * 32);
#pragma unroll
        for (int c = 0; c < 4; ++c)
          dst[c] = make_uint4(pack_bf16(o[c * 8 + 0], o[c * 8 + 1]), pack_bf16(o[c * 8 + 2], o[c * 8 + 3]),
                              pack_bf16(o[c * 8 + 4], o[c * 8 + 5]), pack_bf16(o[c * 8 + 6], o[c * 8 + 7]));
      }
    }
    if (row_ok && part == 0 && P.lse)
      P.lse[((size_t)sg.b * P.Q + r) * P.Hq + sg.g * P.G + hg] = (Mrow + log2f(Lrow)) * kLn2;
  }
  tc_fence_before();
  __syncwarp();
  if (lane == 0) mbar_arrive(bar(BAR_OFREE));
  sc.n += cnt;
  ++sc.seg;
  return true;
}

// ------------------------------------------------------------------------------------------------
// Main kernel
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const TcParams P, const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sm_base = smem_u32(smem);
  const uint32_t bar_base = sm_base + kSmBar;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kSmBar + BAR_COUNT * 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kSmBar + BAR_COUNT * 8 + 8);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x;
  auto bar = [&](int i) { return bar_base + 8u * (uint32_t)i; };

  // ---- setup that touches nothing an earlier kernel wrote (it runs while the K/V append drains): barriers,
  // TMEM, zero the ring (stale V rows of a ragged tile must be finite)
  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) { mbar_init(bar(BAR_FULL + i), 1); mbar_init(bar(BAR_EMPTY + i), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar(BAR_SFULL + i), 1); mbar_init(bar(BAR_PFULL + i), 4); }
    mbar_init(bar(BAR_ODONE), 1);
    mbar_init(bar(BAR_ODONE + 1), 1);
    mbar_init(bar(BAR_OFREE), 4);
    mbar_init(bar(BAR_QFULL), 4);
    *abort_flag = (sm_base & 1023u) ? 1 : 0;  // the swizzled layouts below assume a 1 KiB aligned window
    *reinterpret_cast<volatile unsigned long long*>(abort_flag + 2) = P.wait_ns;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  {
    uint4* z = reinterpret_cast<uint4*>(smem);
    for (int i = threadIdx.x; i < kSmBar / 16; i += kThreads) z[i] = make_uint4(0, 0, 0, 0);
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_async_smem();
  tc_fence_before();
  pdl_wait();               // the block's K/V rows are in the pages from here on
  pdl_launch_dependents();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const int* prefix = P.tile_prefix;
  const int* slot_info = nullptr;
  if (P.B <= kMaxSmemPrefixSlots) {
    int* sm_prefix = reinterpret_cast<int*>(smem + kSmPrefix);
    int* sm_slot = reinterpret_cast<int*>(smem + kSmSlot);
    block_tile_prefix(P, sm_prefix, sm_slot, reinterpret_cast<int*>(smem + kSmMl), cta == 0);
    prefix = sm_prefix;
    slot_info = sm_slot;
  }
  const uint32_t tmem_s0 = tmem + kTmS, tmem_o = tmem + kTmO, tmem_q = tmem + kTmQ;

  if (warp >= 4 && warp < 4 + kProducerWarps) {
    // =========================================================================== TMA producers
    const uint32_t pw = (uint32_t)(warp - 4);  // this warp serves the fills f with f % kProducerWarps == pw
    WorkIter it;
    it.init(P, cta, prefix, slot_info);
    Segment sg;
    uint32_t fill = 0;
    while (it.next(P, cta, sg) && !*abort_flag) {
      const int cnt = sg.j1 - sg.j0;
      const int32_t* pt = P.page_table + (size_t)sg.b * P.max_pages;
      // Page ids are fetched 32 at a time (4 tiles) and one chunk ahead, so that the table lookup is
      // off the critical path of the copies; lane l of a chunk register holds the id of page 32c + l.
      const int total_pages = (sg.kv_len + ISD_PAGE - 1) / ISD_PAGE;
      const int base_page = sg.j0 * 8;
      auto load_chunk = [&](int c) -> int {
        const int pg = base_page + c * 32 + lane;
        int id = 0;
        if (pg < total_pages) id = pt[pg];
        return min(max(id, 0), P.num_pages - 1);
      };
      int cur_c = 0;
      int ids_cur = load_chunk(0), ids_nxt = load_chunk(1);
      // fill order = consumption order: K(0), then for each i: K(i+1), V(i)
      auto issue = [&](int i, bool is_v) -> bool {
        const int j = sg.j0 + i;
        const int valid = min(8, (sg.kv_len - j * kTile + ISD_PAGE - 1) / ISD_PAGE);
        const int src = ((i >> 2) == cur_c) ? ids_cur : ids_nxt;
        const uint32_t s = fill % kStages, ph = (fill / kStages) & 1u;
        if (fill % kProducerWarps == pw) {
          {
            if (!mbar_wait(bar(BAR_EMPTY + s), ph ^ 1u, abort_flag)) return false;
          }
          if (lane == 0) mbar_arrive_expect_tx(bar(BAR_FULL + s), (uint32_t)valid * 4096u);
          __syncwarp();
          const int pg = lane >> 1, half = lane & 1;
          const int pid = __shfl_sync(0xffffffffu, src, ((i & 3) << 3) + (pg & 7));
          if (lane < 16 && pg < valid) {
            const uint32_t dst = sm_base + kSmRing + s * kStageBytes + half * 16384 + pg * 2048;
            tma_load_3d(dst, is_v ? &tmap_v : &tmap_k, half * 64, 0, pid * P.Hkv + sg.g, bar(BAR_FULL + s));
          }
          __syncwarp();
        }
        ++fill;
        if (is_v && (i & 3) == 3) {  // V(i) is the last user of chunk i / 4
          ++cur_c;
          ids_cur = ids_nxt;
          ids_nxt = load_chunk(cur_c + 1);
        }
        return true;
      };
      bool ok = issue(0, false);
      for (int i = 0; i < cnt && ok; ++i) {
        if (i + 1 < cnt) ok = issue(i + 1, false);
        if (ok) ok = issue(i, true);
      }
      if (!ok) break;
    }
    // drain: every issued copy must have landed before the CTA may exit
    // (the consumer waits on every FULL barrier it was promised; on abort wait here, bounded)
    if (*abort_flag) {
      for (uint32_t f = (fill > kStages ? fill - kStages : 0); f < fill; ++f)
        mbar_wait(bar(BAR_FULL + f % kStages), (f / kStages) & 1u, abort_flag);
    }
  } else if (warp == 7) {
    // =========================================================================== MMA issuer
    WorkIter it;
    it.init(P, cta, prefix, slot_info);
    Segment sg;
    uint32_t cons = 0, n = 0, seg = 0;
    const uint32_t idesc_qk = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
    const uint32_t idesc_pv = idesc_qk | (1u << 16);  // B (= V) is MN-major
    bool ok = true;
    while (ok && it.next(P, cta, sg) && !*abort_flag) {
      const int cnt = sg.j1 - sg.j0;
      ok = mbar_wait(bar(BAR_QFULL), seg & 1u, abort_flag);
      if (!ok) break;
      tc_fence_after();
      auto qk = [&](uint32_t nn) -> bool {
        const uint32_t s = cons % kStages, ph = (cons / kStages) & 1u;
        {
          if (!mbar_wait(bar(BAR_FULL + s), ph, abort_flag)) return false;
        }
        // S[nn & 1] is free: QK(nn) follows PV(nn-2) in issue order, and PV(nn-2) was issued only after
        // the softmax warps had read S(nn-2) and stored P(nn-2) over it
        tc_fence_after();
        if (elect_one()) {
          const uint32_t kb = sm_base + kSmRing + s * kStageBytes;
#pragma unroll
          for (int k = 0; k < 8; ++k) {  // 16 dims = 8 packed columns of Q per step
            const uint32_t off = (uint32_t)(k >> 2) * 16384u + (uint32_t)(k & 3) * 32u;
            tc_mma_ts(tmem_s0 + (nn & 1u) * 128u, tmem_q + (seg & 1u) * 64u + (uint32_t)k * 8u, smem_desc(kb + off, 16, 1024), idesc_qk, k > 0);
          }
          tc_commit(bar(BAR_EMPTY + s));
          tc_commit(bar(BAR_SFULL + (nn & 1u)));
        }
        __syncwarp();
        ++cons;
        return true;
      };
      auto pv = [&](uint32_t nn, bool first) -> bool {
        const uint32_t s = cons % kStages, ph = (cons / kStages) & 1u;
        {
          if (!mbar_wait(bar(BAR_FULL + s), ph, abort_flag)) return false;
        }
        {
          if (!mbar_wait(bar(BAR_PFULL + (nn & 1u)), (nn >> 1) & 1u, abort_flag)) return false;
        }
        if (first && seg > 0 && !mbar_wait(bar(BAR_OFREE), (seg - 1u) & 1u, abort_flag)) return false;
        tc_fence_after();
        if (elect_one()) {
          const uint32_t vb = sm_base + kSmRing + s * kStageBytes;
          const uint32_t pt_ = tmem_s0 + (nn & 1u) * 128u;
#pragma unroll
          for (int k = 0; k < 8; ++k)  // 16 keys = 8 packed columns of P per step
            tc_mma_ts(tmem_o, pt_ + (uint32_t)k * 8u, smem_desc(vb + (uint32_t)k * 2048u, 16384, 1024),
                      idesc_pv, !(first && k == 0));
          tc_commit(bar(BAR_EMPTY + s));
          tc_commit(bar(BAR_ODONE + (nn & 1u)));
        }
        __syncwarp();
        ++cons;
        return true;
      };
      ok = qk(n);
      for (int i = 0; i < cnt && ok; ++i) {
        if (i + 1 < cnt) ok = qk(n + i + 1);
        if (ok) ok = pv(n + i, i == 0);
      }
      n += cnt;
      ++seg;
    }
  } else if (warp < 4) {
    // =========================================================================== softmax / epilogue
    WorkIter it;
    it.init(P, cta, prefix, slot_info);
    Segment sg;
    SoftmaxCtx sc;
    sc.smem = smem; sc.bar_base = bar_base; sc.abort_flag = abort_flag;
    sc.tmem_s0 = tmem_s0; sc.tmem_o = tmem_o; sc.tmem_q = tmem_q;
    sc.n = 0; sc.seg = 0;
    bool ok = true;
    Segment sg_next;
    bool have = it.next(P, cta, sg);
    if (have) stage_q(P, sg, sc, 0);
    while (ok && have && !*abort_flag) {
      const bool have_next = it.next(P, cta, sg_next);
      const Segment* nx = have_next ? &sg_next : nullptr;
      const int rows_valid = sg.q_len * P.G;
      if (rows_valid > 64) ok = softmax_segment<1>(P, sg, sc, nx);
      else if (rows_valid > 32) ok = softmax_segment<2>(P, sg, sc, nx);
      else ok = softmax_segment<4>(P, sg, sc, nx);
      sg = sg_next;
      have = have_next;
    }
  }

  // ---- teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicOr(P.global_status, ISD_ST_KERNEL_TIMEOUT);
  if (warp == 4) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
}

// ------------------------------------------------------------------------------------------------
// Combine: pairs whose tiles were split over several CTAs (log-sum-exp merge of the partials)
// ------------------------------------------------------------------------------------------------
// One CTA per share of the main kernel: CTA c merges the pair that starts inside share c and runs on
// into later shares (every split pair has exactly one such share).  The kernel is pure latency (a few
// dependent rounds of small loads), so it is laid out wide: the slot of the share's last tile is found by
// a counting vote over the tile prefix instead of a binary search of dependent loads, and one warp per
// block row merges all partials of its row in a single round.
constexpr int kCombineThreads = 1024;
__global__ void __launch_bounds__(kCombineThreads) attn_combine_kernel(const TcParams P) {
  const int c0 = blockIdx.x;
  pdl_wait();
  pdl_launch_dependents();
  const long long total = (long long)P.tile_prefix[P.B] * P.Hkv;
  if (total == 0) return;
  const long long per = share_units(total, P.num_ctas);
  const long long t_last = ((long long)(c0 + 1) * per < total ? (long long)(c0 + 1) * per : total) - 1;
  if (t_last < (long long)c0 * per) return;  // empty share
  // slot of the share's last tile = number of slots whose tiles all lie at or before t_last
  __shared__ int sm_cnt;
  if (threadIdx.x == 0) sm_cnt = 0;
  __syncthreads();
  {
    int cnt = 0;
    for (int i = threadIdx.x; i < P.B; i += kCombineThreads)
      cnt += ((long long)P.tile_prefix[i + 1] * P.Hkv <= t_last) ? 1 : 0;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
    if ((threadIdx.x & 31) == 0 && cnt) atomicAdd(&sm_cnt, cnt);
  }
  __syncthreads();
  const int b = sm_cnt;
  const int T = P.tile_prefix[b + 1] - P.tile_prefix[b];  // on the split axis: kSegCost units, then the tiles
  const int g = (int)((t_last - (long long)P.tile_prefix[b] * P.Hkv) / T);
  const long long p0 = (long long)P.tile_prefix[b] * P.Hkv + (long long)g * T, p1 = p0 + T;
  const int c_first = (int)((p0 + kSegCost) / per), c_last = (int)((p1 - 1) / per);  // shares that hold tiles of the pair
  if (c_first != c0 || c_last == c0) return;  // merged by an earlier share, or written directly
  const int q_len = P.n_ver[b] + P.N;
  const int rows_valid = q_len * P.G;
  // replicas of a row (key split across lane groups, see softmax_segment) are further partials
  const int F = rows_valid > 64 ? 1 : (rows_valid > 32 ? 2 : 4);
  const int RG = 128 / F;
  const int lane = threadIdx.x & 31;
  const int n_part = (c_last - c_first + 1) * F;  // partials of a row: lane i < n_part fetches the i-th (max, sum)
  for (int row = threadIdx.x >> 5; row < rows_valid; row += kCombineThreads / 32) {
    float M = -INFINITY, L = 0.f, acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int base = 0; base < n_part; base += 32) {
      // one round of loads for up to 32 partials: every lane reads one (max, sum) pair
      float m_i = -INFINITY, l_i = 0.f;
      size_t rr_i = 0;
      if (base + lane < n_part) {
        const int c = c_first + (base + lane) / F, pp = (base + lane) % F;
        const int slot = c * 2 + (((long long)c * per >= p0) ? 0 : 1);
        rr_i = (size_t)slot * 128 + pp * RG + row;
        const float2 ml = *reinterpret_cast<const float2*>(P.part_ml + rr_i * 2);
        m_i = ml.x;
        l_i = ml.y;
      }
      float Mn = m_i;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) Mn = fmaxf(Mn, __shfl_xor_sync(0xffffffffu, Mn, off));
      Mn = fmaxf(Mn, M);
      const float keep = (M == -INFINITY) ? 0.f : ex2f(M - Mn);
      L *= keep;
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[i] *= keep;
      M = Mn;
      const float w_i = (m_i == -INFINITY) ? 0.f : ex2f(m_i - M);
      const int cnt = min(32, n_part - base);
      for (int i = 0; i < cnt; i += 4) {  // four independent loads in flight
        float4 o[4];
        float w[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int ii = min(i + u, cnt - 1);
          const float wu = __shfl_sync(0xffffffffu, w_i, ii);
          const float lu = __shfl_sync(0xffffffffu, l_i, ii);
          const size_t rr = __shfl_sync(0xffffffffu, (unsigned long long)rr_i, ii);
          w[u] = (i + u < cnt) ? wu : 0.f;
          L += lu * w[u];
          o[u] = *reinterpret_cast<const float4*>(P.part_o + rr * 128 + lane * 4);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          acc[0] += o[u].x * w[u]; acc[1] += o[u].y * w[u]; acc[2] += o[u].z * w[u]; acc[3] += o[u].w * w[u];
        }
      }
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
    const int r = row / P.G, hg = row % P.G;
    const size_t o_off = (((size_t)b * P.Q + r) * P.Hq + g * P.G + hg) * ISD_HEAD_DIM + lane * 4;
    *reinterpret_cast<uint2*>(P.out + o_off) = make_uint2(pack_bf16(acc[0] * inv, acc[1] * inv), pack_bf16(acc[2] * inv, acc[3] * inv));
    if (P.lse && lane == 0) P.lse[((size_t)b * P.Q + r) * P.Hq + g * P.G + hg] = (M + log2f(L)) * kLn2;
  }
}

// ------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// pool viewed as [num_pages * Hkv][16 tokens][128 dims]; box = 64 dims x 16 tokens of one (page, head)
int encode_pool_map(CUtensorMap* map, const void* pool, int num_pages, int Hkv) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return ISD_ERR_CUDA;
  const cuuint64_t dims[3] = {ISD_HEAD_DIM, ISD_PAGE, (cuuint64_t)num_pages * (cuuint64_t)Hkv};
  const cuuint64_t strides[2] = {ISD_HEAD_DIM * 2, ISD_HEAD_DIM * 2 * ISD_PAGE};
  const cuuint32_t box[3] = {64, ISD_PAGE, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(pool), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? ISD_OK : ISD_ERR_CUDA;
}

// Tensor maps are encoded once per (k_pool, v_pool) pair and kept: a multi-layer step walks through one pair
// per layer at every call.
constexpr int kMapCacheSize = 128;
struct PoolMaps {
  const void* k_base;
  const void* v_base;
  CUtensorMap map_k, map_v;
};
struct TcHost {
  PoolMaps maps[kMapCacheSize];
  int n_maps, next_victim;
  int* tile_prefix;
};

}  // namespace


int isd_attn_tc_create(isd_ctx* ctx) {
  TcHost* h = new (std::nothrow) TcHost();
  if (!h) return ISD_ERR_NO_MEMORY;
  h->tile_prefix = nullptr;
  h->n_maps = 0;
  h->next_victim = 0;
  ctx->tmap_k = h;
  ctx->attn_ctas = ctx->num_sms;
  if (cudaMalloc(&h->tile_prefix, sizeof(int) * (ctx->cfg.batch + 1)) != cudaSuccess) return ISD_ERR_NO_MEMORY;
  if (cudaMalloc(&ctx->attn_part_o, sizeof(float) * (size_t)ctx->attn_ctas * 2 * 128 * 128) != cudaSuccess) return ISD_ERR_NO_MEMORY;
  if (cudaMalloc(&ctx->attn_part_ml, sizeof(float) * (size_t)ctx->attn_ctas * 2 * 128 * 2) != cudaSuccess) return ISD_ERR_NO_MEMORY;
  if (cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
    return ISD_ERR_CUDA;
  if (!get_encode()) return ISD_ERR_CUDA;
  return ISD_OK;
}

void isd_attn_tc_destroy(isd_ctx* ctx) {
  TcHost* h = reinterpret_cast<TcHost*>(ctx->tmap_k);
  if (h) {
    cudaFree(h->tile_prefix);
    delete h;
  }
  cudaFree(ctx->attn_part_o);
  cudaFree(ctx->attn_part_ml);
  ctx->tmap_k = nullptr;
}

int isd_launch_attn_tc(isd_ctx* ctx, const isd_batch_state* st, const void* q, const void* k_new, const void* v_new,
                       void* k_pool, void* v_pool, void* out, float* lse, cudaStream_t stream) {
  (void)k_new; (void)v_new;  // already appended to the pages by the scatter kernel
  TcHost* h = reinterpret_cast<TcHost*>(ctx->tmap_k);
  if (!h) return ISD_ERR_INVALID_ARG;
  const isd_config& c = ctx->cfg;
  PoolMaps* pm = nullptr;
  for (int i = 0; i < h->n_maps && !pm; ++i)
    if (h->maps[i].k_base == k_pool && h->maps[i].v_base == v_pool) pm = &h->maps[i];
  if (!pm) {
    pm = h->n_maps < kMapCacheSize ? &h->maps[h->n_maps] : &h->maps[h->next_victim];
    int rc = encode_pool_map(&pm->map_k, k_pool, c.num_pages, c.n_kv_heads);
    if (rc == ISD_OK) rc = encode_pool_map(&pm->map_v, v_pool, c.num_pages, c.n_kv_heads);
    if (rc != ISD_OK) {
      pm->k_base = pm->v_base = nullptr;
      return rc;
    }
    pm->k_base = k_pool;
    pm->v_base = v_pool;
    if (h->n_maps < kMapCacheSize) ++h->n_maps;
    else h->next_victim = (h->next_victim + 1) % kMapCacheSize;
  }
  TcParams P;
  P.B = c.batch; P.Q = ctx->Q; P.N = c.stride; P.Hq = c.n_q_heads; P.Hkv = c.n_kv_heads; P.G = ctx->G;
  P.max_pages = c.max_pages_per_slot; P.num_pages = c.num_pages;
  P.scale2 = ctx->sm_scale * kLog2e;
  P.ctx_len = st->ctx_len; P.n_ver = st->n_ver; P.active = st->active; P.page_table = st->page_table;
  P.slot_status = st->slot_status; P.global_status = ctx->global_status;
  P.q = (const __nv_bfloat16*)q; P.out = (__nv_bfloat16*)out; P.lse = lse;
  P.tile_prefix = h->tile_prefix; P.part_o = ctx->attn_part_o; P.part_ml = ctx->attn_part_ml;
  P.num_ctas = ctx->attn_ctas;
  P.wait_ns = ctx->wait_ns;
  cudaError_t e = cudaSuccess;
  if (c.batch > kMaxSmemPrefixSlots) e = isd_launch_pdl(attn_plan_kernel, dim3(1), dim3(1024), 0, stream, P);
  if (ctx->ev_attn0) cudaEventRecord(ctx->ev_attn0, stream);
  if (e == cudaSuccess)
    e = isd_launch_pdl(attn_tc_kernel, dim3(ctx->attn_ctas), dim3(kThreads), kSmemBytes, stream, P, pm->map_k, pm->map_v);
  if (ctx->ev_attn1) cudaEventRecord(ctx->ev_attn1, stream);
  if (e == cudaSuccess) e = isd_launch_pdl(attn_combine_kernel, dim3(ctx->attn_ctas), dim3(kCombineThreads), 0, stream, P);
  ctx->launches += 2 + (c.batch > kMaxSmemPrefixSlots ? 1 : 0);
  return e == cudaSuccess ? ISD_OK : ISD_ERR_CUDA;
}
