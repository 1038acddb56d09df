// isd_lora_linear: segment-gated LoRA linear layer of the lossless R-ISD variant (Sec. 3.2, the R-ISD
// paragraph and Eq. 5): y_j = W x_j + 1[j in MASK] * s * B A x_j over the M = B * Q token rows of a step.
//
// One tcgen05 GEMM kernel (C = A1 B1^T (+ A2 B2^T), bf16 operands, fp32 accumulation in tensor memory) computes
//   t = gate * s * (x A^T)            [M, R]  the gated, scaled down-projection (bf16), and
//   y = x W^T + t B^T                 [M, N]  one GEMM over the two K segments (K, then R)
// so the gate costs nothing in the large GEMM and clean rows provably see the base weights only (their t is 0).
// In one launch when rank <= 256 or a multiple of 256: the last CTAs first compute one 128-row x (<= 256)-column
// block of t each and publish it (a counter per row block, raised after a proxy fence: t is read back by TMA);
// the producer of an output tile waits (bounded) until the counter of its row block is complete before it loads
// the second K segment, which comes last.
// The last CTA to finish clears the flags.  Otherwise two launches of the same kernel, t first.  The output tiles
// of the last, partial round of the grid are cut into column strips, one per CTA.
//
// Two forms of the kernel.  gemm_tc2_kernel (further down, the one normally used) works on CTA pairs; the one-CTA
// form below serves shapes the pairs cannot take (ranks above 256 that are not multiples of 256, more blocks of t
// than CTA pairs).
//
// One-CTA kernel: persistent CTAs, one 128 x BN output tile at a time.  Warp 4 streams the operands with TMA
// (2-D maps, 64-element K slices = 128-byte rows, SWIZZLE_128B, every CTA loads for itself) into a 4-stage ring; warp 5
// issues tcgen05.mma (M = 128, N = BN, K = 16, both operands from shared memory) into one of two TMEM
// accumulators; warps 0-3 read the other accumulator back (tcgen05.ld, one lane = one row), apply gate and
// scale, and store bf16, so the epilogue of a tile overlaps the main loop of the next.  Every mbarrier wait is
// bounded (status bit 0x80000000, then the CTA drains and frees its tensor memory).
#include <cuda.h>
#include <cuda_bf16.h>

#include "isd_internal.cuh"
#include "isd_lora_work.cuh"

namespace {

constexpr int kThreads = 192;
constexpr int kBM = 128;
constexpr int kBK = 64;                       // bf16 elements per K slice = one 128-byte swizzled row
constexpr int kStages = 4;                    // 4 x 48 KiB ring of the one-CTA kernel

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
// Bounded wait: false (and the abort flag raised) when the time limit is reached or somebody else gave up.
// The limit (nanoseconds) sits in shared memory two words behind the abort flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long budget = *reinterpret_cast<const volatile unsigned long long*>(abort_flag + 2);
  return isd_bounded_wait(budget, abort_flag, [&]() { return mbar_try_wait(bar, parity); });
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
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
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accum) : "memory");
}
// K-major shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1: rows of 128 bytes, groups of
// eight rows 1024 bytes apart
__device__ __forceinline__ uint64_t smem_desc_kmajor(uint32_t addr) {
  const uint32_t lo = ((addr & 0x3FFFFu) >> 4) | ((16u >> 4) << 16);
  const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
  return ((uint64_t)hi << 32) | lo;
}
#define TMEM_LD32(taddr, v)                                                                             \
  asm volatile(                                                                                         \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                         \
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25," \
      "%26,%27,%28,%29,%30,%31}, [%32];"                                                                \
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), \
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]),        \
        "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]),      \
        "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]),      \
        "=r"(v[29]), "=r"(v[30]), "=r"(v[31])                                                           \
      : "r"(taddr))
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

struct GemmParams {
  int M, N, K1, K2;           // C[M, N] = A1[M, K1] B1[N, K1]^T + A2[M, K2] B2[N, K2]^T   (K2 = 0: one segment)
  __nv_bfloat16* c;           // row-major, leading dimension N
  const uint8_t* gate;        // [M] or nullptr: rows with gate 0 are written as zeros
  float scale;
  uint32_t* global_status;
  // fused down-projection (fuse != 0): the last tiles_m * t_chunks CTAs first compute one 128-row x Rc-column
  // block each of t[M, R] = t_gate * t_scale * (A1 Bt^T), Bt[R, K1], and publish it; the second K segment of C
  // (A2 = t) waits until all t_chunks blocks of its rows are there
  int fuse, R, Rc, t_chunks;  // Rc = columns of a block of t (R = t_chunks * Rc)
  int tail_split;             // the tiles of the last, partial round are cut into this many column strips (1, 2 or 4)
  __nv_bfloat16* t;
  const uint8_t* t_gate;
  float t_scale;
  uint32_t* flags;            // [tiles_m] blocks of t written for that row block (all zero between launches)
  uint32_t* done;             // [1] CTAs that have finished (zero between launches)
  unsigned long long wait_ns; // time limit of a device-side wait
};

__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// orders accesses through the generic proxy (ordinary loads and stores) with those of the async proxy (TMA)
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }

enum { BAR_FULL = 0, BAR_EMPTY = kStages, BAR_ACC_FULL = 2 * kStages, BAR_ACC_FREE = 2 * kStages + 2,
       BAR_COUNT = 2 * kStages + 4 };

template <int BN>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const GemmParams P, const __grid_constant__ CUtensorMap map_a1, const __grid_constant__ CUtensorMap map_b1,
               const __grid_constant__ CUtensorMap map_a2, const __grid_constant__ CUtensorMap map_b2,
               const __grid_constant__ CUtensorMap map_bt, const __grid_constant__ CUtensorMap map_b1n,
               const __grid_constant__ CUtensorMap map_b2n) {
  constexpr int kStageA = kBM * kBK * 2, kStageB = BN * kBK * 2, kStageBytes = kStageA + kStageB;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sm_base = smem_u32(smem);
  const uint32_t bar_base = sm_base + kStages * kStageBytes;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kStages * kStageBytes + BAR_COUNT * 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kStages * kStageBytes + BAR_COUNT * 8 + 8);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  auto bar = [&](int i) { return bar_base + 8u * (uint32_t)i; };
  if (sm_base & 1023u) {  // the swizzled layout assumes a 1 KiB aligned window
    if (threadIdx.x == 0) atomicOr(P.global_status, ISD_ST_KERNEL_TIMEOUT);
    return;
  }
  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) { mbar_init(bar(BAR_FULL + i), 1); mbar_init(bar(BAR_EMPTY + i), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar(BAR_ACC_FULL + i), 1); mbar_init(bar(BAR_ACC_FREE + i), 4); }
    *abort_flag = 0;
    *reinterpret_cast<volatile unsigned long long*>(abort_flag + 2) = P.wait_ns;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  const int ks1 = P.K1 / kBK, ks2 = P.K2 / kBK, ks = ks1 + ks2;  // K slices per tile
  // Work items of this CTA (isd_lora_work.cuh): assigned by the mirrored block index, so that the blocks of t fall
  // to the lowest block indices; the readers' bounded wait below needs no co-residency of the whole grid.
  LoraWork work;
  work.init((int)blockIdx.x, (int)gridDim.x, P.M, P.N, kBM, BN, P.fuse, P.t_chunks, P.Rc, P.tail_split);
  const int tiles_m = work.tiles_m, n_items = work.n_items, t_block = work.t_block;
  using Item = LoraWorkItem;
  auto item = [&](int it) { return work.item(it); };

  if (warp == 4) {
    // ============================================================================ TMA producer
    uint32_t fill = 0;
    for (int it = 0; it < n_items && !*abort_flag; ++it) {
      const Item w = item(it);
      const bool pre = w.pre, narrow = !pre && w.cols != BN;
      const int m0 = w.m0, n0 = w.n0;
      const int n_slices = pre ? ks1 : ks;
      const uint32_t bytes = (uint32_t)(kStageA + w.cols * kBK * 2);
      bool ok = true;
      for (int i = 0; i < n_slices && ok; ++i, ++fill) {
        const uint32_t s = fill % kStages, ph = (fill / kStages) & 1u;
        ok = mbar_wait(bar(BAR_EMPTY + s), ph ^ 1u, abort_flag);
        if (!ok) break;
        const bool seg2 = !pre && i >= ks1;
        if (P.fuse && seg2 && i == ks1) {
          // the second segment reads t: wait (bounded in time) until this row block of it has been published.
          // Its producers are the CTAs with the lowest block indices, which never wait before they publish.
          ok = isd_bounded_wait(P.wait_ns, abort_flag, [&]() { return ld_acquire(P.flags + m0 / kBM) == (uint32_t)P.t_chunks; });
          if (!ok) break;
          fence_proxy_async();
        }
        if (elect_one()) {
          mbar_arrive_expect_tx(bar(BAR_FULL + s), bytes);  // out-of-range rows are zero-filled, still counted
          const uint32_t dst = sm_base + s * kStageBytes;
          const int k0 = (seg2 ? i - ks1 : i) * kBK;
          tma_load_2d(dst, seg2 ? &map_a2 : &map_a1, k0, m0, bar(BAR_FULL + s));
          tma_load_2d(dst + kStageA, pre ? &map_bt : (seg2 ? (narrow ? &map_b2n : &map_b2) : (narrow ? &map_b1n : &map_b1)), k0, n0,
                      bar(BAR_FULL + s));
        }
        __syncwarp();
      }
      if (!ok) break;
    }
    if (*abort_flag) {  // every issued copy must land before the CTA may leave
      for (uint32_t f = (fill > kStages ? fill - kStages : 0); f < fill; ++f)
        mbar_wait(bar(BAR_FULL + f % kStages), (f / kStages) & 1u, abort_flag);
    }
  } else if (warp == 5) {
    // ============================================================================ MMA issuer
    auto idesc_for = [](int n) { return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24); };
    uint32_t cons = 0, t_local = 0;
    for (int it = 0; it < n_items && !*abort_flag; ++it, ++t_local) {
      const Item w = item(it);
      const bool pre = w.pre;
      const int n_slices = pre ? ks1 : ks;
      const uint32_t idesc = idesc_for(w.cols);
      const uint32_t acc = t_local & 1u;
      // the epilogue warps must have read this accumulator's previous tile
      if (t_local >= 2 && !mbar_wait(bar(BAR_ACC_FREE + acc), ((t_local >> 1) - 1u) & 1u, abort_flag)) break;
      tc_fence_after();
      bool ok = true;
      for (int i = 0; i < n_slices && ok; ++i, ++cons) {
        const uint32_t s = cons % kStages, ph = (cons / kStages) & 1u;
        ok = mbar_wait(bar(BAR_FULL + s), ph, abort_flag);
        if (!ok) break;
        tc_fence_after();
        if (elect_one()) {
          const uint32_t a0 = sm_base + s * kStageBytes, b0 = a0 + kStageA;
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k)
            tc_mma(tmem + acc * (uint32_t)BN, smem_desc_kmajor(a0 + k * 32), smem_desc_kmajor(b0 + k * 32),
                   idesc, (i > 0 || k > 0) ? 1u : 0u);
          tc_commit(bar(BAR_EMPTY + s));
          if (i == n_slices - 1) tc_commit(bar(BAR_ACC_FULL + acc));
        }
        __syncwarp();
      }
      if (!ok) break;
    }
  } else {
    // ============================================================================ epilogue (warps 0-3)
    uint32_t t_local = 0;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    for (int it = 0; it < n_items && !*abort_flag; ++it, ++t_local) {
      const Item w = item(it);
      const bool pre = w.pre;
      const int m0 = w.m0, n0 = w.n0;
      const int n_cols = w.cols, ld_c = pre ? P.R : P.N, n_lim = pre ? P.R : P.N;
      __nv_bfloat16* c = pre ? P.t : P.c;
      const uint8_t* gate = pre ? P.t_gate : P.gate;
      const uint32_t acc = t_local & 1u;
      if (!mbar_wait(bar(BAR_ACC_FULL + acc), (t_local >> 1) & 1u, abort_flag)) break;
      tc_fence_after();
      const int row = m0 + warp * 32 + lane;
      const bool row_ok = row < P.M;
      const float f = (gate == nullptr || (row_ok && gate[row])) ? (pre ? P.t_scale : P.scale) : 0.f;
#pragma unroll 1
      for (int c0 = 0; c0 < n_cols; c0 += 32) {
        uint32_t v[32];
        TMEM_LD32(tmem + lane_base + acc * (uint32_t)BN + (uint32_t)c0, v);
        tmem_wait_ld();
        if (row_ok && n0 + c0 < n_lim) {  // the column counts are multiples of 32 here (checked by the launcher)
          uint4* dst = reinterpret_cast<uint4*>(c + (size_t)row * ld_c + n0 + c0);
#pragma unroll
          for (int q = 0; q < 4; ++q)
            dst[q] = make_uint4(pack_bf16(__uint_as_float(v[8 * q]) * f, __uint_as_float(v[8 * q + 1]) * f),
                                pack_bf16(__uint_as_float(v[8 * q + 2]) * f, __uint_as_float(v[8 * q + 3]) * f),
                                pack_bf16(__uint_as_float(v[8 * q + 4]) * f, __uint_as_float(v[8 * q + 5]) * f),
                                pack_bf16(__uint_as_float(v[8 * q + 6]) * f, __uint_as_float(v[8 * q + 7]) * f));
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_ACC_FREE + acc));
      if (pre) {
        // publish the block of t: every epilogue thread's stores, made visible to the TMA reads of other CTAs
        fence_proxy_async();
        __threadfence();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (threadIdx.x == 0) atomicAdd(P.flags + t_block, 1u);  // after the fence above: a release
      }
    }
  }
  // ---- teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicOr(P.global_status, ISD_ST_KERNEL_TIMEOUT);
  if (P.fuse && threadIdx.x == 0) {  // the CTA that finishes last leaves the flags as it found them
    __threadfence();
    if (atomicAdd(P.done, 1u) == gridDim.x - 1) {
      for (int m = 0; m < tiles_m; ++m) P.flags[m] = 0u;
      *P.done = 0u;
    }
  }
  if (warp == 4) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
}

// ------------------------------------------------------------------------------------------------
// The same GEMM on CTA pairs (tcgen05 cta_group::2): a cluster of two CTAs owns a 256 x 256 output tile.  Each CTA
// stages its own 128 rows of A and 128 of the tile's 256 rows of B (half the shared-memory traffic per flop of the
// one-CTA form), the first CTA of the pair issues M = 256 MMAs that read both CTAs' shared memory and write both
// CTAs' tensor memory (rows 0-127 into its own, 128-255 into its partner's), and each CTA's epilogue warps store
// their 128 rows.  Barriers: TMA of both CTAs reports to the first CTA's `full` barrier; the MMA thread's commits
// arrive on the `empty` and `accumulator full` barriers of both CTAs; the epilogue warps of both CTAs arrive on
// the first CTA's `accumulator free` barrier.  Every wait is bounded.
// ------------------------------------------------------------------------------------------------
constexpr int kStages2 = 6;
constexpr int kStage2A = kBM * kBK * 2, kStage2B = 128 * kBK * 2, kStage2Bytes = kStage2A + kStage2B;
constexpr int kBN2 = 256;
enum { B2_FULL = 0, B2_EMPTY = kStages2, B2_ACC_FULL = 2 * kStages2, B2_ACC_FREE = 2 * kStages2 + 2,
       B2_COUNT = 2 * kStages2 + 4 };

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// the address, in the cluster's shared window, of this CTA's shared-memory address `addr` in CTA `rank`
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load of a CTA pair: the bytes land in this CTA's shared memory and are reported to the barrier at `bar`,
// an address in the cluster's shared window (the first CTA's barrier)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t cluster_addr) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accum) : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_tc2_kernel(const GemmParams P, const __grid_constant__ CUtensorMap map_a1, const __grid_constant__ CUtensorMap map_b1,
                const __grid_constant__ CUtensorMap map_a2, const __grid_constant__ CUtensorMap map_b2,
                const __grid_constant__ CUtensorMap map_bt, const __grid_constant__ CUtensorMap map_b1n,
                const __grid_constant__ CUtensorMap map_b2n) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sm_base = smem_u32(smem);
  const uint32_t bar_base = sm_base + kStages2 * kStage2Bytes;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kStages2 * kStage2Bytes + B2_COUNT * 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kStages2 * kStage2Bytes + B2_COUNT * 8 + 8);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();
  const bool leader = rank == 0;
  auto bar = [&](int i) { return bar_base + 8u * (uint32_t)i; };
  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages2; ++i) { mbar_init(bar(B2_FULL + i), 1); mbar_init(bar(B2_EMPTY + i), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar(B2_ACC_FULL + i), 1); mbar_init(bar(B2_ACC_FREE + i), 8); }
    *abort_flag = (sm_base & 1023u) ? 1 : 0;  // the swizzled layout assumes a 1 KiB aligned window
    *reinterpret_cast<volatile unsigned long long*>(abort_flag + 2) = P.wait_ns;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {  // the same warp in both CTAs
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the partner's barriers exist before anything is reported to them
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  const int ks1 = P.K1 / kBK, ks2 = P.K2 / kBK, ks = ks1 + ks2;
  // work items of the pair (isd_lora_work.cuh), by the mirrored pair index: a block of t first, whole tiles, one
  // column strip
  LoraWork work;
  work.init((int)blockIdx.x >> 1, (int)gridDim.x >> 1, P.M, P.N, 2 * kBM, kBN2, P.fuse, P.t_chunks, P.Rc, P.tail_split);
  const int tiles_m = work.tiles_m, n_items = work.n_items, t_block = work.t_block;
  using Item = LoraWorkItem;
  auto item = [&](int it) { return work.item(it); };

  if (warp == 4) {
    // ============================================================================ TMA producer (both CTAs)
    uint32_t fill = 0;
    for (int it = 0; it < n_items && !*abort_flag; ++it) {
      const Item w = item(it);
      const bool pre = w.pre, narrow = !pre && w.cols != kBN2;
      const int m0 = w.m0 + (int)rank * kBM;          // this CTA's rows of A
      const int half = w.cols / 2, n0 = w.n0 + (int)rank * half;  // this CTA's rows of B
      const int n_slices = pre ? ks1 : ks;
      const uint32_t bytes = 2u * (uint32_t)(kStage2A + half * kBK * 2);  // of both CTAs
      bool ok = true;
      for (int i = 0; i < n_slices && ok; ++i, ++fill) {
        const uint32_t s = fill % kStages2, ph = (fill / kStages2) & 1u;
        ok = mbar_wait(bar(B2_EMPTY + s), ph ^ 1u, abort_flag);
        if (!ok) break;
        const bool seg2 = !pre && i >= ks1;
        if (P.fuse && seg2 && i == ks1) {
          // bounded in time; the producers of t are the pairs with the lowest block indices (see above)
          ok = isd_bounded_wait(P.wait_ns, abort_flag,
                                [&]() { return ld_acquire(P.flags + w.m0 / (2 * kBM)) == 2u * (uint32_t)P.t_chunks; });
          if (!ok) break;
          fence_proxy_async();
        }
        if (elect_one()) {
          const uint32_t full = map_to_cta(bar(B2_FULL + s), 0u);
          if (leader) mbar_arrive_expect_tx(bar(B2_FULL + s), bytes);
          const uint32_t dst = sm_base + s * kStage2Bytes;
          const int k0 = (seg2 ? i - ks1 : i) * kBK;
          tma_load_2d_pair(dst, seg2 ? &map_a2 : &map_a1, k0, m0, full);
          tma_load_2d_pair(dst + kStage2A, pre ? &map_bt : (seg2 ? (narrow ? &map_b2n : &map_b2) : (narrow ? &map_b1n : &map_b1)), k0, n0, full);
        }
        __syncwarp();
      }
      if (!ok) break;
    }
    if (*abort_flag && leader) {  // every issued copy must land before the CTAs may leave
      for (uint32_t f = (fill > kStages2 ? fill - kStages2 : 0); f < fill; ++f)
        mbar_wait(bar(B2_FULL + f % kStages2), (f / kStages2) & 1u, abort_flag);
    }
  } else if (warp == 5) {
    // ============================================================================ MMA issuer (first CTA only)
    if (leader) {
      auto idesc_for = [](int n) { return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)((2 * kBM) >> 4) << 24); };
      uint32_t cons = 0, t_local = 0;
      for (int it = 0; it < n_items && !*abort_flag; ++it, ++t_local) {
        const Item w = item(it);
        const int n_slices = w.pre ? ks1 : ks;
        const uint32_t idesc = idesc_for(w.cols);
        const uint32_t acc = t_local & 1u;
        if (t_local >= 2 && !mbar_wait(bar(B2_ACC_FREE + acc), ((t_local >> 1) - 1u) & 1u, abort_flag)) break;
        tc_fence_after();
        bool ok = true;
        for (int i = 0; i < n_slices && ok; ++i, ++cons) {
          const uint32_t s = cons % kStages2, ph = (cons / kStages2) & 1u;
          ok = mbar_wait(bar(B2_FULL + s), ph, abort_flag);
          if (!ok) break;
          tc_fence_after();
          if (elect_one()) {
            const uint32_t a0 = sm_base + s * kStage2Bytes, b0 = a0 + kStage2A;
#pragma unroll
            for (int k = 0; k < kBK / 16; ++k)
              tc_mma_pair(tmem + acc * (uint32_t)kBN2, smem_desc_kmajor(a0 + k * 32), smem_desc_kmajor(b0 + k * 32), idesc,
                          (i > 0 || k > 0) ? 1u : 0u);
            tc_commit_pair(map_to_cta(bar(B2_EMPTY + s), 0u));
            tc_commit_pair(map_to_cta(bar(B2_EMPTY + s), 1u));
            if (i == n_slices - 1) {
              tc_commit_pair(map_to_cta(bar(B2_ACC_FULL + acc), 0u));
              tc_commit_pair(map_to_cta(bar(B2_ACC_FULL + acc), 1u));
            }
          }
          __syncwarp();
        }
        if (!ok) break;
      }
    }
  } else {
    // ============================================================================ epilogue (warps 0-3, both CTAs)
    uint32_t t_local = 0;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    for (int it = 0; it < n_items && !*abort_flag; ++it, ++t_local) {
      const Item w = item(it);
      const bool pre = w.pre;
      const int m0 = w.m0 + (int)rank * kBM, n0 = w.n0;
      const int n_cols = w.cols, ld_c = pre ? P.R : P.N, n_lim = pre ? P.R : P.N;
      __nv_bfloat16* c = pre ? P.t : P.c;
      const uint8_t* gate = pre ? P.t_gate : P.gate;
      const uint32_t acc = t_local & 1u;
      if (!mbar_wait(bar(B2_ACC_FULL + acc), (t_local >> 1) & 1u, abort_flag)) break;
      tc_fence_after();
      const int row = m0 + warp * 32 + lane;
      const bool row_ok = row < P.M;
      const float f = (gate == nullptr || (row_ok && gate[row])) ? (pre ? P.t_scale : P.scale) : 0.f;
#pragma unroll 1
      for (int c0 = 0; c0 < n_cols; c0 += 32) {
        uint32_t v[32];
        TMEM_LD32(tmem + lane_base + acc * (uint32_t)kBN2 + (uint32_t)c0, v);
        tmem_wait_ld();
        if (row_ok && n0 + c0 < n_lim) {
          uint4* dst = reinterpret_cast<uint4*>(c + (size_t)row * ld_c + n0 + c0);
#pragma unroll
          for (int q = 0; q < 4; ++q)
            dst[q] = make_uint4(pack_bf16(__uint_as_float(v[8 * q]) * f, __uint_as_float(v[8 * q + 1]) * f),
                                pack_bf16(__uint_as_float(v[8 * q + 2]) * f, __uint_as_float(v[8 * q + 3]) * f),
                                pack_bf16(__uint_as_float(v[8 * q + 4]) * f, __uint_as_float(v[8 * q + 5]) * f),
                                pack_bf16(__uint_as_float(v[8 * q + 6]) * f, __uint_as_float(v[8 * q + 7]) * f));
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_cta(bar(B2_ACC_FREE + acc), 0u));
      if (pre) {
        fence_proxy_async();
        __threadfence();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (threadIdx.x == 0) atomicAdd(P.flags + t_block, 1u);  // after the fence above: a release
      }
    }
  }
  // ---- teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicOr(P.global_status, ISD_ST_KERNEL_TIMEOUT);
  if (P.fuse && threadIdx.x == 0) {  // the CTA that finishes last leaves the flags as it found them
    __threadfence();
    if (atomicAdd(P.done, 1u) == gridDim.x - 1) {
      for (int m = 0; m < tiles_m; ++m) P.flags[m] = 0u;
      *P.done = 0u;
    }
  }
  cluster_sync_all();  // nobody frees tensor memory or leaves while the partner may still use this CTA's
  if (warp == 4) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
}

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

// row-major bf16 matrix [rows, cols] viewed in boxes of 64 columns x box_rows rows
int encode_matrix(CUtensorMap* map, const void* base, int rows, int cols, int box_rows) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return ISD_ERR_CUDA;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? ISD_OK : ISD_ERR_CUDA;
}

constexpr int kMaxFlags = 4096;  // row blocks of t that the fused kernel can track

template <int BN>
int launch_gemm(isd_ctx* ctx, GemmParams P, const void* a1, const void* b1, const void* a2, const void* b2,
                const void* bt, cudaStream_t stream) {
  constexpr int kSmem = kStages * (kBM * kBK * 2 + BN * kBK * 2) + BAR_COUNT * 8 + 64;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(gemm_tc_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) != cudaSuccess)
      return ISD_ERR_CUDA;
    attr_set = true;
  }
  CUtensorMap ma1, mb1, ma2, mb2, mbt, mb1n, mb2n;
  int rc = encode_matrix(&ma1, a1, P.M, P.K1, kBM);
  if (rc == ISD_OK) rc = encode_matrix(&mb1, b1, P.N, P.K1, BN);
  if (rc == ISD_OK) rc = P.K2 ? encode_matrix(&ma2, a2, P.M, P.K2, kBM) : encode_matrix(&ma2, a1, P.M, P.K1, kBM);
  if (rc == ISD_OK) rc = P.K2 ? encode_matrix(&mb2, b2, P.N, P.K2, BN) : encode_matrix(&mb2, b1, P.N, P.K1, BN);
  if (rc == ISD_OK) rc = P.fuse ? encode_matrix(&mbt, bt, P.R, P.K1, P.Rc) : encode_matrix(&mbt, b1, P.N, P.K1, BN);
  if (rc != ISD_OK) return rc;
  // grid and column strips of the last, partial round (isd_lora_work.cuh)
  int grid;
  lora_grid(P.M, P.N, kBM, BN, P.fuse, P.t_chunks, ctx->num_sms, true, grid, P.tail_split);
  rc = encode_matrix(&mb1n, b1, P.N, P.K1, BN / P.tail_split);
  if (rc == ISD_OK) rc = P.K2 ? encode_matrix(&mb2n, b2, P.N, P.K2, BN / P.tail_split) : encode_matrix(&mb2n, b1, P.N, P.K1, BN / P.tail_split);
  if (rc != ISD_OK) return rc;
  gemm_tc_kernel<BN><<<grid, kThreads, kSmem, stream>>>(P, ma1, mb1, ma2, mb2, mbt, mb1n, mb2n);
  ctx->launches++;
  return cudaGetLastError() == cudaSuccess ? ISD_OK : ISD_ERR_CUDA;
}

// The CTA-pair form: same arguments; fuse, R, Rc, t_chunks as prepared by the caller (blocks of t are 256 rows here).
int launch_gemm_pair(isd_ctx* ctx, GemmParams P, const void* a1, const void* b1, const void* a2, const void* b2,
                     const void* bt, cudaStream_t stream) {
  constexpr int kSmem = kStages2 * kStage2Bytes + B2_COUNT * 8 + 64;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(gemm_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) != cudaSuccess)
      return ISD_ERR_CUDA;
    attr_set = true;
  }
  int pairs;
  lora_grid(P.M, P.N, 2 * kBM, kBN2, P.fuse, P.t_chunks, ctx->num_sms / 2, false, pairs, P.tail_split);
  const int strip_half = kBN2 / P.tail_split / 2;
  CUtensorMap ma1, mb1, ma2, mb2, mbt, mb1n, mb2n;
  int rc = encode_matrix(&ma1, a1, P.M, P.K1, kBM);
  if (rc == ISD_OK) rc = encode_matrix(&mb1, b1, P.N, P.K1, kBN2 / 2);
  if (rc == ISD_OK) rc = P.K2 ? encode_matrix(&ma2, a2, P.M, P.K2, kBM) : encode_matrix(&ma2, a1, P.M, P.K1, kBM);
  if (rc == ISD_OK) rc = P.K2 ? encode_matrix(&mb2, b2, P.N, P.K2, kBN2 / 2) : encode_matrix(&mb2, b1, P.N, P.K1, kBN2 / 2);
  if (rc == ISD_OK) rc = P.fuse ? encode_matrix(&mbt, bt, P.R, P.K1, P.Rc / 2) : encode_matrix(&mbt, b1, P.N, P.K1, kBN2 / 2);
  if (rc == ISD_OK) rc = encode_matrix(&mb1n, b1, P.N, P.K1, strip_half);
  if (rc == ISD_OK) rc = P.K2 ? encode_matrix(&mb2n, b2, P.N, P.K2, strip_half) : encode_matrix(&mb2n, b1, P.N, P.K1, strip_half);
  if (rc != ISD_OK) return rc;
  gemm_tc2_kernel<<<2 * pairs, kThreads, kSmem, stream>>>(P, ma1, mb1, ma2, mb2, mbt, mb1n, mb2n);
  ctx->launches++;
  return cudaGetLastError() == cudaSuccess ? ISD_OK : ISD_ERR_CUDA;
}

}  // namespace

int isd_lora_create(isd_ctx* ctx) {
  if (cudaMalloc(&ctx->lora_flags, sizeof(uint32_t) * (kMaxFlags + 1)) != cudaSuccess) return ISD_ERR_NO_MEMORY;
  return cudaMemset(ctx->lora_flags, 0, sizeof(uint32_t) * (kMaxFlags + 1)) == cudaSuccess ? ISD_OK : ISD_ERR_CUDA;
}

void isd_lora_destroy(isd_ctx* ctx) {
  cudaFree(ctx->lora_flags);
  ctx->lora_flags = nullptr;
}

// Width of an output tile of the one-CTA kernel = widest MMA (N = 256): the fewest B-panel re-reads per flop.
constexpr int kLoraBN = 256;

int isd_launch_lora_linear(isd_ctx* ctx, const isd_lora_args* a, cudaStream_t stream) {
  GemmParams P2;
  P2.M = a->m; P2.N = a->n; P2.K1 = a->k; P2.K2 = a->rank;
  P2.c = reinterpret_cast<__nv_bfloat16*>(a->y); P2.gate = nullptr; P2.scale = 1.f;
  P2.global_status = ctx->global_status;
  P2.fuse = 0; P2.R = a->rank; P2.Rc = a->rank; P2.t_chunks = 1; P2.t = reinterpret_cast<__nv_bfloat16*>(a->t); P2.t_gate = a->gate; P2.t_scale = a->scale;
  P2.flags = ctx->lora_flags; P2.done = ctx->lora_flags + kMaxFlags;
  P2.wait_ns = ctx->wait_ns;
  // One launch when t divides into blocks of one MMA's width (rank <= the tile width, or a multiple of it) and
  // every block gets its own CTA: the last CTAs compute t = gate * scale * (x A^T) block by block before their
  // output tiles, and the second K segment of y = x W^T + t B^T waits for the blocks of the rows it reads.
  const LoraPlan plan = lora_plan(a->m, a->n, a->rank, ctx->num_sms, kMaxFlags);
  if (plan.form == 2) {
    // CTA pairs: 256 x 256 tiles, blocks of t of 256 rows
    P2.fuse = 1;
    P2.t_chunks = plan.t_chunks;
    P2.Rc = plan.Rc;
    return launch_gemm_pair(ctx, P2, a->x, a->w, a->t, a->b, a->a, stream);
  }
  if (plan.form == 1) {
    P2.fuse = 1;
    P2.t_chunks = plan.t_chunks;
    P2.Rc = plan.Rc;
    return launch_gemm<kLoraBN>(ctx, P2, a->x, a->w, a->t, a->b, a->a, stream);
  }
  // Otherwise two launches.  1. t = gate * scale * (x A^T): N = rank, one K segment
  GemmParams P1 = P2;
  P1.N = a->rank; P1.K2 = 0; P1.c = reinterpret_cast<__nv_bfloat16*>(a->t); P1.gate = a->gate; P1.scale = a->scale;
  int rc = launch_gemm<128>(ctx, P1, a->x, a->a, nullptr, nullptr, nullptr, stream);
  if (rc != ISD_OK) return rc;
  // 2. y = x W^T + t B^T: two K segments, no gate (it is already in t)
  return launch_gemm<kLoraBN>(ctx, P2, a->x, a->w, a->t, a->b, nullptr, stream);
}

// Host-only view of the work assignment (no GPU needed): what unit `unit_index` of the launch that writes y does as
// its item `item`.  out = {form, units, items of this unit, pre, m0, n0, cols, tile rows, tile columns}.
extern "C" int isd_test_lora_work_item(int32_t m, int32_t n, int32_t rank, int32_t num_sms, int32_t unit_index, int32_t item,
                                       int32_t* out) {
  if (!out || m < 1 || n < 1 || rank < 1 || num_sms < 2) return ISD_ERR_INVALID_ARG;
  const LoraPlan p = lora_plan(m, n, rank, num_sms, kMaxFlags);
  if (unit_index < 0 || unit_index >= p.units) return ISD_ERR_INVALID_ARG;
  LoraWork w;
  w.init(unit_index, p.units, m, n, p.bm, p.bn, p.fuse, p.t_chunks, p.Rc, p.tail_split);
  out[0] = p.form; out[1] = p.units; out[2] = w.n_items; out[7] = p.bm; out[8] = p.bn;
  out[3] = out[4] = out[5] = out[6] = -1;
  if (item >= 0 && item < w.n_items) {
    const LoraWorkItem it = w.item(item);
    out[3] = it.pre; out[4] = it.m0; out[5] = it.n0; out[6] = it.cols;
  }
  return ISD_OK;
}
