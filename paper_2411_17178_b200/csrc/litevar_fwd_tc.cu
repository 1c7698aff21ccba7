// Tensor-core forward kernel for sm_100a: TMA-staged bf16 tiles, tcgen05 MMAs with TMEM
// accumulators, fp32 online softmax, element mask from the plan's bit blocks.
//
// One CTA handles one (query tile, head, batch row) and walks the live key tiles of its query
// tile in plan order.  Warp roles:
//   warp 0      TMA producer (one lane): Q once, then K and V of every live key tile into a ring
//   warp 1      TMEM allocation; one lane issues S = Q K^T and O += P V
//   warps 2..5  softmax: thread = query row (TMEM lane); mask, running max/sum, P -> TMEM (bf16),
//               O rescale when the row max moves, final normalise + store (twice under CFG sharing)
// TMEM columns: S fp32 [0,128), O fp32 [128,192), P bf16x2 [192,256).
//
// Every wait is bounded: when a wait runs out the CTA raises the plan's status word, drains its
// outstanding copies, frees its TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <mutex>

#include "litevar_internal.h"

namespace litevar {

namespace {

constexpr int kStages = 2;
constexpr int kThreads = 192;
constexpr uint32_t kTileBytes = kBlockN * kHeadDim * 2;  // 16 KB: 128 rows of 128 B
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t kColS = 0, kColO = 128, kColP = 192;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s

struct SharedStorage {
  alignas(1024) uint8_t q[kTileBytes];
  alignas(1024) uint8_t k[kStages][kTileBytes];
  alignas(1024) uint8_t v[kStages][kTileBytes];
  alignas(8) uint64_t bar_q;
  uint64_t bar_k[kStages];
  uint64_t bar_v[kStages];
  uint64_t bar_free[kStages];
  uint64_t bar_s;
  uint64_t bar_p;
  uint64_t bar_o;
  uint32_t tmem_base;
  int abort_flag;
};

// Instruction descriptors (kind::f16): D fp32, A/B bf16, M = 128.
//   bits 4-5 D format (1 = f32), 7-9 A format (1 = bf16), 10-12 B format (1 = bf16),
//   bit 15 A major (0 = K), bit 16 B major (0 = K, 1 = MN), bits 17-22 N >> 3, bits 24-28 M >> 4.
constexpr uint32_t kIdescQK = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBlockN >> 3) << 17) |
                              ((uint32_t)(kBlockM >> 4) << 24);
constexpr uint32_t kIdescPV = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) |
                              ((uint32_t)(kHeadDim >> 3) << 17) | ((uint32_t)(kBlockM >> 4) << 24);

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Shared-memory matrix descriptor for a tile of 128-byte rows written by TMA with the 128-byte
// swizzle: 8-row groups are 1024 B apart (stride byte offset); version 1; layout type 2 = SWIZZLE_128B.
// The same encoding serves a K-major operand (Q, K: rows = M/N index, 64 contiguous K elements) and the
// MN-major V operand (rows = keys = K index, 64 contiguous N elements).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr) {
  return (uint64_t)((saddr >> 4) & 0x3FFFu) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
         (2ull << 61);
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
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          int32_t* status) {
  if (mbar_try(bar, parity)) return true;
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

__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(smem_u32(bar))
      : "memory");
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
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
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
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
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
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

__global__ void __launch_bounds__(kThreads, 2)
fwd_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
              const __grid_constant__ CUtensorMap tm_v, FwdParams p) {
  extern __shared__ uint8_t smem_raw[];
  SharedStorage& sm = *reinterpret_cast<SharedStorage*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const SetDesc sd = p.sets[p.head_to_set ? p.head_to_set[h] : 0];
  const int pair_begin = sd.row_ptr[qt];
  const int n_tiles = sd.row_ptr[qt + 1] - pair_begin;
  volatile int* abort_flag = &sm.abort_flag;

  if (threadIdx.x == 0) {
    mbar_init(&sm.bar_q, 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sm.bar_k[s], 1);
      mbar_init(&sm.bar_v[s], 1);
      mbar_init(&sm.bar_free[s], 1);
    }
    mbar_init(&sm.bar_s, 1);
    mbar_init(&sm.bar_p, 128);
    mbar_init(&sm.bar_o, 1);
    sm.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp == 0) {
    if (lane == 0 && n_tiles > 0) {
      // ---------------------------------------------------------------- TMA producer
      mbar_expect_tx(&sm.bar_q, kTileBytes);
      tma_load_4d(sm.q, &tm_q, 0, qt * kBlockM, h, b, &sm.bar_q);
      int issued = 0;
      for (int i = 0; i < n_tiles; ++i) {
        const int s = i % kStages, n = i / kStages;
        if (n > 0 && !mbar_wait(&sm.bar_free[s], (uint32_t)((n - 1) & 1), abort_flag, p.status)) break;
        const int t0 = sd.pairs[pair_begin + i].key_tile * kBlockN;
        mbar_expect_tx(&sm.bar_k[s], kTileBytes);
        tma_load_4d(sm.k[s], &tm_k, 0, t0, h, b, &sm.bar_k[s]);
        mbar_expect_tx(&sm.bar_v[s], kTileBytes);
        tma_load_4d(sm.v[s], &tm_v, 0, t0, h, b, &sm.bar_v[s]);
        issued = i + 1;
      }
      if (*abort_flag) {
        // wait (bounded) for copies still in flight before the CTA may exit
        (void)mbar_wait(&sm.bar_q, 0u, abort_flag, p.status);
        for (int i = issued > kStages ? issued - kStages : 0; i < issued; ++i) {
          const int s = i % kStages, n = i / kStages;
          const unsigned long long t0 = global_ns();
          while (!(mbar_try(&sm.bar_k[s], (uint32_t)(n & 1)) && mbar_try(&sm.bar_v[s], (uint32_t)(n & 1))))
            if (global_ns() - t0 > kWaitLimitNs) break;
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && n_tiles > 0) {
      // ---------------------------------------------------------------- MMA issuer
      const uint64_t q_desc = make_desc(smem_u32(sm.q));
      bool ok = mbar_wait(&sm.bar_q, 0u, abort_flag, p.status);
      for (int i = 0; ok && i < n_tiles; ++i) {
        const int s = i % kStages;
        const uint32_t ph = (uint32_t)((i / kStages) & 1);
        if (!(ok = mbar_wait(&sm.bar_k[s], ph, abort_flag, p.status))) break;
        tc_fence_after();
        const uint64_t k_desc = make_desc(smem_u32(sm.k[s]));
#pragma unroll
        for (int kk = 0; kk < kHeadDim / 16; ++kk)  // 16 bf16 = 32 B per step inside the swizzle row
          mma_ss(tmem + kColS, q_desc + 2 * kk, k_desc + 2 * kk, kIdescQK, kk > 0 ? 1u : 0u);
        mma_commit(&sm.bar_s);
        if (!(ok = mbar_wait(&sm.bar_p, (uint32_t)(i & 1), abort_flag, p.status))) break;
        if (!(ok = mbar_wait(&sm.bar_v[s], ph, abort_flag, p.status))) break;
        tc_fence_after();
        const uint64_t v_desc = make_desc(smem_u32(sm.v[s]));
#pragma unroll
        for (int kk = 0; kk < kBlockN / 16; ++kk)  // 16 keys = 16 rows of 128 B = 2048 B; P: 8 packed columns
          mma_ts(tmem + kColO, tmem + kColP + 8 * kk, v_desc + (uint64_t)(2048 >> 4) * kk, kIdescPV,
                 (i > 0 || kk > 0) ? 1u : 0u);
        mma_commit(&sm.bar_free[s]);
        if (i == n_tiles - 1) mma_commit(&sm.bar_o);
      }
    }
  } else if (n_tiles > 0) {
    // ------------------------------------------------------------------ softmax + epilogue
    const int lane_group = warp & 3;  // TMEM lanes this warp may touch: 32*lane_group .. +31
    const int m = lane_group * 32 + lane;
    const int q = qt * kBlockM + m;
    const uint32_t tbase = tmem + ((uint32_t)(lane_group * 32) << 16);
    const float sc = p.sm_scale * 1.4426950408889634f;
    float row_max = -INFINITY, row_sum = 0.f;
    bool ok = true;
    uint32_t r[32];
    for (int i = 0; i < n_tiles; ++i) {
      const Pair pr = sd.pairs[pair_begin + i];
      uint4 bits4 = make_uint4(~0u, ~0u, ~0u, ~0u);
      if (pr.mask_block >= 0) bits4 = sd.mask[(size_t)pr.mask_block * kBlockM + m];
      const uint32_t bits[4] = {bits4.x, bits4.y, bits4.z, bits4.w};
      if (!(ok = mbar_wait(&sm.bar_s, (uint32_t)(i & 1), abort_flag, p.status))) break;
      tc_fence_after();
      // pass 1: row maximum over live keys
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        tmem_ld32(tbase + kColS + 32 * c, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e)
          if ((bits[c] >> e) & 1u) mx = fmaxf(mx, __uint_as_float(r[e]));
      }
      const float new_max = fmaxf(row_max, mx);
      const float alpha = row_max == -INFINITY ? 1.f : exp2f((row_max - new_max) * sc);
      const float msc = new_max == -INFINITY ? 0.f : new_max * sc;
      if (i > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          tmem_ld32(tbase + kColO + 32 * c, r);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
          tmem_st32(tbase + kColO + 32 * c, r);
        }
      }
      // pass 2: probabilities, row sum (from unrounded p), P as packed bf16 into TMEM
      float psum = 0.f;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        tmem_ld32(tbase + kColS + 32 * c, r);
        tmem_wait_ld();
        uint32_t pk[16];
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          float p0 = ((bits[c] >> e) & 1u) ? exp2f(fmaf(__uint_as_float(r[e]), sc, -msc)) : 0.f;
          float p1 = ((bits[c] >> (e + 1)) & 1u) ? exp2f(fmaf(__uint_as_float(r[e + 1]), sc, -msc)) : 0.f;
          psum += p0 + p1;
          pk[e >> 1] = pack_bf16(p0, p1);
        }
        tmem_st16(tbase + kColP + 16 * c, pk);
      }
      row_sum = row_sum * alpha + psum;
      row_max = new_max;
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&sm.bar_p);
    }
    if (ok && (ok = mbar_wait(&sm.bar_o, 0u, abort_flag, p.status))) {
      tc_fence_after();
      const float inv = 1.f / row_sum;
      uint16_t* orow = p.out + (int64_t)b * p.o_sb + (int64_t)h * p.o_sh + (int64_t)q * p.o_st;
      uint16_t* orow2 = orow + (int64_t)p.share_offset * p.o_sb;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        tmem_ld32(tbase + kColO + 32 * c, r);
        tmem_wait_ld();
        if (q < p.n_k) {
#pragma unroll
          for (int e = 0; e < 32; e += 8) {
            uint4 o4;
            o4.x = pack_bf16(__uint_as_float(r[e + 0]) * inv, __uint_as_float(r[e + 1]) * inv);
            o4.y = pack_bf16(__uint_as_float(r[e + 2]) * inv, __uint_as_float(r[e + 3]) * inv);
            o4.z = pack_bf16(__uint_as_float(r[e + 4]) * inv, __uint_as_float(r[e + 5]) * inv);
            o4.w = pack_bf16(__uint_as_float(r[e + 6]) * inv, __uint_as_float(r[e + 7]) * inv);
            *reinterpret_cast<uint4*>(orow + 32 * c + e) = o4;
            if (p.share_offset > 0) *reinterpret_cast<uint4*>(orow2 + 32 * c + e) = o4;
          }
        }
      }
    }
  }

  // ---------------------------------------------------------------------- teardown (all paths)
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

// ------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
    else
      (void)cudaGetLastError();
  });
  return fn;
}

// Rank-4 map over a [batch, head, token, 64] bf16 tensor with element strides; box = 128 tokens x 64.
bool encode_map(CUtensorMap* tm, const void* base, int64_t rows, int64_t heads, int64_t batch, int64_t st,
                int64_t sh, int64_t sb) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  // a dimension of extent 1 may come with any stride; give it a valid one
  if (heads == 1 && sh < kHeadDim) sh = st * rows;
  if (batch == 1 && sb < kHeadDim) sb = sh * heads;
  cuuint64_t gdim[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)rows, (cuuint64_t)heads, (cuuint64_t)batch};
  cuuint64_t gstr[3] = {(cuuint64_t)st * 2, (cuuint64_t)sh * 2, (cuuint64_t)sb * 2};
  cuuint32_t box[4] = {(cuuint32_t)kHeadDim, (cuuint32_t)kBlockN, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), gdim, gstr, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace

litevar_status_t launch_forward_tcgen05(const FwdParams& p, int n_q_tiles, cudaStream_t stream) {
  static std::once_flag attr_once;
  static cudaError_t attr_err = cudaSuccess;
  constexpr int smem_bytes = (int)sizeof(SharedStorage) + 1024;
  std::call_once(attr_once, [] {
    attr_err = cudaFuncSetAttribute(fwd_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  });
  if (attr_err != cudaSuccess) return LITEVAR_ERR_CUDA;
  CUtensorMap tm_q, tm_k, tm_v;
  if (!encode_map(&tm_q, p.q, p.n_k, p.n_heads, p.batch_computed, p.q_st, p.q_sh, p.q_sb) ||
      !encode_map(&tm_k, p.k, p.L_k, p.n_heads, p.batch_computed, p.k_st, p.k_sh, p.k_sb) ||
      !encode_map(&tm_v, p.v, p.L_k, p.n_heads, p.batch_computed, p.v_st, p.v_sh, p.v_sb))
    return LITEVAR_ERR_INVALID_ARG;
  dim3 grid((unsigned)n_q_tiles, (unsigned)p.n_heads, (unsigned)p.batch_computed);
  fwd_tc_kernel<<<grid, kThreads, smem_bytes, stream>>>(tm_q, tm_k, tm_v, p);
  if (cudaGetLastError() != cudaSuccess) return LITEVAR_ERR_CUDA;
  return LITEVAR_OK;
}

}  // namespace litevar
