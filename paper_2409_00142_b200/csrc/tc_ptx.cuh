// Inline-PTX wrappers and constants shared by the kernels that run the LM head on the sm_100a
// tensor cores: mbarriers with bounded waits, bulk / tensor copies, tcgen05 MMA, commit and
// tensor-memory loads, shared-memory and instruction descriptors.
#pragma once

#include <cuda.h>

#include "ddd_common.cuh"

namespace ddd {
namespace tc {

constexpr int kEpiWarps = 16;           // warps 2..17: four of them read tensor memory, all fold rows
constexpr int kEpiThreads = 32 * kEpiWarps;
constexpr int kTcThreads = 64 + kEpiThreads;
constexpr int kBlockM = 128;            // vocab rows per MMA tile
constexpr int kBlockK = 64;             // hidden elements per stage: one 128-byte swizzle row
constexpr int kUmmaK = 16;              // K of one tcgen05.mma with 16-bit operands
constexpr int kUnitRows = 32;           // vocab rows per TMA box of W
constexpr int kUnitBytes = kUnitRows * kBlockK * 2;   // 4096
constexpr int kABytes = kBlockM * kBlockK * 2;        // 16384
constexpr int kChunkCols = 16;          // accumulator columns (beam rows) per epilogue chunk
constexpr int kSmemLimit = 232448;      // 227 KB opt-in limit per block
constexpr unsigned long long kWaitLimitNs = 2000000000ull;
constexpr int kL2PrefetchBytes = 128 * 1024;   // per block, ahead of the dependency wait (at most 148 blocks: about 19 MB in all)


// ---------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ unsigned long long global_timer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if the wait ran out of time (limit_ns by %globaltimer) or another
// role already gave up; a wait that runs out records DDD_ERR_TIMEOUT and raises the block's flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                          bool heed_abort = true, unsigned long long limit_ns = kWaitLimitNs) {
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 1023u) {
      if (heed_abort && *abort_flag) return false;
      const unsigned long long now = global_timer();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) {
        atomicCAS(status, DDD_OK, DDD_ERR_TIMEOUT);
        *abort_flag = 1;
        return false;
      }
    }
  }
}
__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.b32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ int ld_relaxed_gpu(const int* p) {
  int v;
  asm volatile("ld.relaxed.gpu.global.b32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// Grid-wide hand-over: waits until *counter >= target (every block adds one per hand-over; the
// counters only grow during a launch).  False if the wait ran out - DDD_ERR_TIMEOUT is recorded
// and the grid-wide abort word raised - or another block gave up.
__device__ __forceinline__ bool grid_wait(const int* counter, int target, int* abort_word, int* status,
                                          unsigned long long limit_ns = kWaitLimitNs) {
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (ld_acquire_gpu(counter) >= target) return true;
    if ((it & 15u) == 15u) {
      if (ld_relaxed_gpu(abort_word) != 0) return false;
      const unsigned long long now = global_timer();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) {
        atomicCAS(status, DDD_OK, DDD_ERR_TIMEOUT);
        atomicExch(abort_word, 1);
        return false;
      }
    }
  }
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
      : "memory");
}
// Plain (untiled) bulk copy global -> shared; addresses and size are multiples of 16 bytes.
__device__ __forceinline__ void bulk_load_hint(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar,
                                               unsigned long long policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy)
      : "memory");
}
// Asks L2 to fetch a contiguous region (multiple of 16 bytes); nothing lands in shared memory.
__device__ __forceinline__ void l2_prefetch(const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, unsigned long long a_desc, unsigned long long b_desc,
                                            uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_load_16cols(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_load_8cols(uint32_t taddr, float (&v)[8]) {
  uint32_t r[8];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x8.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void epilogue_barrier() {
  asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
}
// Barrier over the epilogue threads that also ANDs a flag, so that all their warps take the
// same decision after a bounded wait.
__device__ __forceinline__ bool epilogue_all(bool ok) {
  uint32_t r;
  asm volatile(
      "{\n"
      ".reg .pred p, q;\n"
      "setp.ne.b32 p, %1, 0;\n"
      "bar.red.and.pred q, 1, %2, p;\n"
      "selp.u32 %0, 1, 0, q;\n"
      "}\n"
      : "=r"(r)
      : "r"(ok ? 1u : 0u), "n"(kEpiThreads)
      : "memory");
  return r != 0;
}

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 bf16) wide
// and 128-byte swizzled: 8-row groups are 1024 bytes apart (stride byte offset); the leading
// byte offset is not used by swizzled K-major layouts.  Bits: [0,14) address >> 4,
// [16,30) LBO >> 4, [32,46) SBO >> 4, [46,48) version 1, [61,64) layout 2 = SWIZZLE_128B.
__device__ __forceinline__ unsigned long long make_smem_desc(uint32_t addr) {
  return (unsigned long long)((addr & 0x3FFFFu) >> 4) | (1ull << 16) | ((unsigned long long)(1024 >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// Instruction descriptor for kind::f16: D = f32 (bits [4,6) = 1), A = B = bf16 (bits [7,10)
// and [10,13) = 1), both K-major (bits 15, 16 = 0), N >> 3 at [17,23), M >> 4 at [24,29).
__device__ __forceinline__ uint32_t make_instr_desc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kBlockM >> 4) << 24);
}

// ---------------------------------------------------------------------------- shared-memory plan
// Accumulator chunks (of kChunkCols beam rows) the epilogue can take out of tensor memory at a
// time: one per group of four epilogue warps, each of which reads one lane quarter.
__host__ __device__ inline int epi_group(int R) {
  const int n_chunks = (R + kChunkCols - 1) / kChunkCols;
  return n_chunks < kEpiWarps / 4 ? n_chunks : kEpiWarps / 4;
}

struct SmemPlan {
  int a, b, zt, key, ms, plant, live, bars, tmem_ptr, abort_flag, total;
};

// Keys kept per beam row in shared memory: k for beams of up to 32 (one key per lane), else k
// rounded up to whole lanes of four (the wide-list layout).
__host__ __device__ inline int key_stride(int k) { return k <= kNarrowK ? k : (k + 3) & ~3; }

// a_units: 32-row units of W a stage holds per K-block (4 = one tile; 5-8 when a block feeds both of its tiles
// from one fetch of h)
__host__ __device__ inline SmemPlan smem_plan(int stages, int ksub, int n_pad, int R, int k, int cpg, int a_units = 4) {
  SmemPlan s;
  int off = 0;
  s.a = off; off += stages * ksub * a_units * kUnitBytes;
  s.b = off; off += stages * ksub * n_pad * kBlockK * 2;
  s.zt = off; off += cpg * kChunkCols * kTile * 4;
  s.key = off; off += R * key_stride(k) * 8;
  s.ms = off; off += R * 8;
  s.plant = off; off += R * 4;
  s.live = off; off += R * 4;
  off = (off + 7) / 8 * 8;
  s.bars = off; off += (2 * stages + 5) * 8;
  s.tmem_ptr = off; off += 4;
  s.abort_flag = off; off += 4;
  s.total = off;
  return s;
}

}  // namespace tc
}  // namespace ddd
