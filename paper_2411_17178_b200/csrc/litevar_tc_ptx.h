// Device-side building blocks of the tensor-core forward kernels (sm_100a): mbarrier, TMA, tcgen05 and TMEM
// wrappers in inline PTX, the shared-memory and instruction descriptors, the tensor maps of one launch and the
// walk over the union of two live key-tile lists.  Included by the forward kernels only.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "litevar_internal.h"

namespace litevar {
namespace tc {

constexpr uint32_t kTileBytes = kBlockN * kHeadDim * 2;  // 16 KB: 128 rows of 128 B
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s
constexpr int kNoTile = 0x7fffffff;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Shared-memory matrix descriptor for a tile of 128-byte rows written by TMA with the 128-byte
// swizzle: 8-row groups are 1024 B apart (stride byte offset); version 1; layout type 2 = SWIZZLE_128B.
// The same encoding serves a K-major operand (Q, K: rows = M/N index, 64 contiguous K elements) and the
// MN-major V operand (rows = keys = K index, 64 contiguous N elements).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr) {
  return (uint64_t)((saddr >> 4) & 0x3FFFu) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
         (2ull << 61);
}
// MN-major operand wider than one 64-element block: the leading-dimension byte offset (bits 16-29)
// is the distance from the first block of N columns to the next one.
__device__ __forceinline__ uint64_t make_desc_mn(uint32_t saddr, uint32_t next_block_bytes) {
  return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)((next_block_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try(uint64_t* bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return done;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait.  Returns false when another role gave up or the time limit passed; the caller then
// leaves its loop and falls through to the common teardown.
__device__ __forceinline__ bool mbar_wait_loop(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                               int32_t* status) {
  const unsigned long long t0 = global_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try(bar, parity)) return true;
    if ((it & 63u) == 0u) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        atomicExch(status, 1);
        return false;
      }
    }
  }
}
static __device__ __noinline__ bool mbar_wait_slow(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                                   int32_t* status) {
  return mbar_wait_loop(bar, parity, abort_flag, status);
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          int32_t* status) {
  if (mbar_try(bar, parity)) return true;
  if (mbar_try(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag, status);
}
// The same wait without a function call (a kernel that moves registers between its warpgroups with setmaxnreg
// cannot call a function compiled for one register count) and with a cheap clock: a few polls first, then
// polls against the SM's cycle counter (the global timer costs hundreds of cycles per read).  The limit is
// 2^32 cycles, two seconds or more at any clock the part runs at.
__device__ __forceinline__ bool mbar_wait_inl(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                              int32_t* status) {
#pragma unroll 1
  for (int it = 0; it < 16; ++it)
    if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
#pragma unroll 1
  for (uint32_t it = 1;; ++it) {
    if (mbar_try(bar, parity)) return true;
    if ((it & 63u) == 0u) {
      if (*abort_flag) return false;
      if (clock64() - t0 > (1ll << 32)) {
        *abort_flag = 1;
        atomicExch(status, 1);
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(smem_u32(bar))
      : "memory");
}

__device__ __forceinline__ void tma_load_5d(void* dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, int c4,
                                            uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(smem_u32(bar))
      : "memory");
}
// Tensor maps of one launch.  q is rank 4 (raster query tiles) or rank 5 (patch query tiles); kr/vr
// cover the raster prefix of the cache; k2/v2[i] cover the grid of the i-th key scale tiled in patches.
struct TensorMaps {
  CUtensorMap q, kr, vr;
  CUtensorMap k2[kMaxPatchScales], v2[kMaxPatchScales];
};

// Loads of one query / key tile according to its geometry.
__device__ __forceinline__ void load_q_tile(void* dst, const TensorMaps& tm, const FwdParams& p, int qt, int h, int b,
                                            uint64_t* bar) {
  if (p.q_geom == nullptr) {
    tma_load_4d(dst, &tm.q, 0, qt * kBlockM, h, b, bar);
    return;
  }
  const TileGeom g = p.q_geom[qt];
  if (g.scale < 0)
    tma_load_4d(dst, &tm.q, 0, g.a, h, b, bar);
  else
    tma_load_5d(dst, &tm.q, 0, g.b, g.a, h, b, bar);
}
__device__ __forceinline__ void load_kv_tile(void* dst, const CUtensorMap* raster, const CUtensorMap* patch,
                                             const FwdParams& p, int kt, int h, int b, uint64_t* bar) {
  if (p.key_geom == nullptr) {
    tma_load_4d(dst, raster, 0, kt * kBlockN, h, b, bar);
    return;
  }
  const TileGeom g = p.key_geom[kt];
  if (g.scale < 0)
    tma_load_4d(dst, raster, 0, g.a, h, b, bar);
  else
    tma_load_5d(dst, patch + g.map_slot, 0, g.b, g.a, h, b, bar);
}

__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Four consecutive K = 16 steps of one product in a single instruction sequence: step i reads A at
// a_tmem + i * kAStep (TMEM columns) and B at b_desc + i * kBStep (descriptor units of 16 bytes); the first step
// accumulates only when `accumulate_first` is non-zero, the others always do.  The issuing lane's own
// instruction stream is what a product of small MMAs waits for (the tensor pipe takes 50 to 65 cycles per step
// at N <= 128, a step issued through per-step address arithmetic and predicate set-up costs two to three times
// that), so the offsets are immediates and nothing but the four MMAs depends on anything.
template <int kA1, int kA2, int kA3, int kB1, int kB2, int kB3>
__device__ __forceinline__ void mma_ts_x4_at(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate_first) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t.reg .b64 b1, b2, b3;\n\t.reg .b32 a1, a2, a3;\n\t"
      "setp.ne.b32 p, %4, 0;\n\tsetp.ne.b32 q, 1, 0;\n\t"
      "add.u32 a1, %1, %5;\n\tadd.u32 a2, %1, %6;\n\tadd.u32 a3, %1, %7;\n\t"
      "add.s64 b1, %2, %8;\n\tadd.s64 b2, %2, %9;\n\tadd.s64 b3, %2, %10;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a1], b1, %3, q;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a2], b2, %3, q;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a3], b3, %3, q;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate_first), "n"(kA1), "n"(kA2), "n"(kA3),
        "n"(kB1), "n"(kB2), "n"(kB3)
      : "memory");
}
template <int kAStep, int kBStep>
__device__ __forceinline__ void mma_ts_x4(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate_first) {
  mma_ts_x4_at<kAStep, 2 * kAStep, 3 * kAStep, kBStep, 2 * kBStep, 3 * kBStep>(d_tmem, a_tmem, b_desc, idesc,
                                                                               accumulate_first);
}
// The same with both operands in shared memory (descriptors).
template <int kAStep, int kBStep>
__device__ __forceinline__ void mma_ss_x4(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate_first) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t.reg .b64 a1, a2, a3, b1, b2, b3;\n\t"
      "setp.ne.b32 p, %4, 0;\n\tsetp.ne.b32 q, 1, 0;\n\t"
      "add.s64 a1, %1, %5;\n\tadd.s64 a2, %1, %6;\n\tadd.s64 a3, %1, %7;\n\t"
      "add.s64 b1, %2, %8;\n\tadd.s64 b2, %2, %9;\n\tadd.s64 b3, %2, %10;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], a1, b1, %3, q;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], a2, b2, %3, q;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], a3, b3, %3, q;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate_first), "n"(kAStep), "n"(2 * kAStep),
        "n"(3 * kAStep), "n"(kBStep), "n"(2 * kBStep), "n"(3 * kBStep)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t* r) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// Launch order of the tensor-core kernels.  The (batch row, head) units are taken in groups of
// p.units_per_group; inside a group the CTAs go query-tile pair by pair (heaviest first, the planner's order), all
// units of the group side by side.  The K/V of one group is what the CTAs resident at one time read: the host
// sizes the group so that it fits in half of L2, and every K/V tile then comes from DRAM once per step instead of
// once per wave of CTAs.
__device__ __forceinline__ void cta_work(const FwdParams& p, int n_ranks, int& rank, int& unit) {
  const int n_units = p.n_heads * p.batch_computed;
  const int g_units = p.units_per_group;
  const int group = blockIdx.x / (g_units * n_ranks);
  const int r = blockIdx.x - group * (g_units * n_ranks);
  const int here = min(g_units, n_units - group * g_units);  // the last group may be smaller
  rank = r / here;
  unit = group * g_units + (r - rank * here);
}

// Walk of the union of two ascending key-tile lists (the two halves of the CTA).
struct UnionWalk {
  const Pair* pairs;
  int i0, e0, i1, e1;
  int kt0, kt1;  // heads of the two lists (kNoTile when exhausted)
  __device__ __forceinline__ void init(const Pair* p, int b0, int end0, int b1, int end1) {
    pairs = p;
    i0 = b0; e0 = end0; i1 = b1; e1 = end1;
    kt0 = i0 < e0 ? __ldg(&pairs[i0].key_tile) : kNoTile;
    kt1 = i1 < e1 ? __ldg(&pairs[i1].key_tile) : kNoTile;
  }
  __device__ __forceinline__ bool has() const { return kt0 != kNoTile || kt1 != kNoTile; }
  // Next key tile and which halves list it; heads are refilled at once so that the loads overlap
  // the caller's waits.
  __device__ __forceinline__ int next(bool& live0, bool& live1) {
    const int kt = min(kt0, kt1);
    live0 = kt0 == kt;
    live1 = kt1 == kt;
    if (live0) kt0 = ++i0 < e0 ? __ldg(&pairs[i0].key_tile) : kNoTile;
    if (live1) kt1 = ++i1 < e1 ? __ldg(&pairs[i1].key_tile) : kNoTile;
    return kt;
  }
};

}  // namespace tc

// Fills the tensor maps of a launch from its parameters (host).  False when an encoding fails.
bool encode_tensor_maps(const FwdParams& p, tc::TensorMaps* tm);

}  // namespace litevar
