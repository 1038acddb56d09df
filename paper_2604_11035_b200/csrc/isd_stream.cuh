// Streaming of logits rows through shared memory, shared by the verification kernels: a ring of
// kRowStages x kRowStageBytes that one thread of a producer warp fills with bulk copies (mbarrier
// full / empty pairs, waits bounded in time) and 256 worker threads read back as 16-byte vectors.
#pragma once
#include "isd_internal.cuh"

namespace {

constexpr int kThreads = 256;  // worker threads of a verification CTA (a producer warp comes on top)

// Eight consecutive logits as fp32 from their raw 16-byte vectors (bf16: byte permutes and masks, which
// run on the ALU pipe; shifts would be issued as integer multiplies on the busier FMA pipe).
template <int DT>
__device__ __forceinline__ void unpack8(const uint4& a, const uint4& b, float (&l)[8]) {
  if (DT == ISD_LOGITS_BF16) {
    l[0] = __uint_as_float(__byte_perm(a.x, 0u, 0x1044)); l[1] = __uint_as_float(a.x & 0xFFFF0000u);
    l[2] = __uint_as_float(__byte_perm(a.y, 0u, 0x1044)); l[3] = __uint_as_float(a.y & 0xFFFF0000u);
    l[4] = __uint_as_float(__byte_perm(a.z, 0u, 0x1044)); l[5] = __uint_as_float(a.z & 0xFFFF0000u);
    l[6] = __uint_as_float(__byte_perm(a.w, 0u, 0x1044)); l[7] = __uint_as_float(a.w & 0xFFFF0000u);
  } else {
    l[0] = __uint_as_float(a.x); l[1] = __uint_as_float(a.y); l[2] = __uint_as_float(a.z); l[3] = __uint_as_float(a.w);
    l[4] = __uint_as_float(b.x); l[5] = __uint_as_float(b.y); l[6] = __uint_as_float(b.z); l[7] = __uint_as_float(b.w);
  }
}

// Eight consecutive logits starting at element e (e % 8 == 0), straight from global memory.
template <int DT>
__device__ __forceinline__ void load8(const void* row, int e, float (&l)[8]) {
  uint4 a, b = make_uint4(0u, 0u, 0u, 0u);
  if (DT == ISD_LOGITS_BF16) {
    a = ld_stream_16B(reinterpret_cast<const uint16_t*>(row) + e);
  } else {
    a = ld_stream_16B(reinterpret_cast<const float*>(row) + e);
    b = ld_stream_16B(reinterpret_cast<const float*>(row) + e + 4);
  }
  unpack8<DT>(a, b, l);
}

constexpr int kRowStages = 4;            // row pass: bulk-copy ring of kRowStages x kRowStageBytes
constexpr int kRowStageBytes = 8192;

// Barrier of the kThreads worker threads (a producer warp, where a kernel has one, stays out of it).
__device__ __forceinline__ void worker_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory"); }

// Order-preserving map float <-> signed int (an involution), so that a warp can agree on a maximum with
// one integer reduction.
__device__ __forceinline__ int ord_key(float f) {
  const int b = __float_as_int(f);
  return b ^ ((b >> 31) & 0x7FFFFFFF);
}
__device__ __forceinline__ float ord_val(int k) { return __int_as_float(k ^ ((k >> 31) & 0x7FFFFFFF)); }

__device__ __forceinline__ float max8(const float (&l)[8]) {
  return fmaxf(max3(l[0], l[1], l[2]), max3(max3(l[3], l[4], l[5]), l[6], l[7]));
}


// Shared memory of the row pass: the ring and its barriers.
struct RowRing {
  __align__(128) unsigned char stage[kRowStages][kRowStageBytes];
  __align__(8) uint64_t full[kRowStages];   // a stage's bytes have landed (one arrival + transaction bytes)
  __align__(8) uint64_t empty[kRowStages];  // every worker warp has read the stage (one arrival per warp)
};

// Producer (one thread): streams bytes [byte_lo, byte_hi) of a row into the ring, one contiguous bulk copy
// per stage.  c is the ring's running stage counter: it carries on over consecutive ranges, so that several
// ranges can go through one ring without re-initialising its barriers.  Returns false when a wait ran out.
__device__ __forceinline__ bool row_producer(RowRing& R, const char* row, size_t byte_lo, size_t byte_hi, int& c,
                                             unsigned long long wait_ns) {
  const uint32_t full0 = ring_smem_u32(R.full), empty0 = ring_smem_u32(R.empty), st0 = ring_smem_u32(R.stage);
  for (size_t off = byte_lo; off < byte_hi; off += kRowStageBytes, ++c) {
    const int s = c & (kRowStages - 1);
    const uint32_t ph = (c / kRowStages) & 1;
    if (!ring_mbar_wait(empty0 + 8 * s, ph ^ 1, wait_ns)) return false;
    const size_t left = byte_hi - off;
    const uint32_t bytes = left < (size_t)kRowStageBytes ? (uint32_t)left : (uint32_t)kRowStageBytes;
    ring_mbar_expect_tx(full0 + 8 * s, bytes);
    ring_bulk_g2s(st0 + s * kRowStageBytes, row + off, bytes, full0 + 8 * s);
  }
  return true;
}

__device__ __forceinline__ bool row_producer(RowRing& R, const char* row, size_t byte_lo, size_t byte_hi,
                                             unsigned long long wait_ns) {
  int c = 0;
  return row_producer(R, row, byte_lo, byte_hi, c, wait_ns);
}


}  // namespace
