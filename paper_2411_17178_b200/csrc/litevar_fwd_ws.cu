// Warp-specialised tensor-core forward kernel for sm_100a with register reallocation: one softmax thread owns a
// whole query row, and the scores of the next key tile are formed while the softmax of the current one runs.
// Used for steps with long tile lists (from eight key tiles per query tile on); the kernel of litevar_fwd_tc.cu
// serves the shorter ones.
//
// The kernel is written for NH query tiles ("halves", 128 queries each) of one (head, batch row) per CTA, walking
// the union of their live key-tile lists; the library launches NH = 1, two CTAs per SM (see launch_forward_ws).
//   warps 0 .. 4 NH - 1   softmax warpgroup of half h = warp / 4: thread m of the group owns query slot m (TMEM
//                         lane m).  A key tile is taken in two passes of 64 keys through one rolled copy of the
//                         code: 64 scores from TMEM into registers, the plan's element mask, the row maximum
//                         without any exchange, the probabilities against a lazily updated reference maximum
//                         (every fourth pair of exponentials on the FMA pipe by a cubic, the rest on the
//                         exponential pipe), their sum, and P (packed bf16) into a TMEM block of its own.  The S
//                         block is released as soon as the second pass has its scores in registers.  At the end
//                         the thread normalises and stores its output row.
//   warp 4 NH             TMA producer (one lane): Q of every half, then K and V of every listed key tile into two
//                         rings of kStages tiles.
//   warp 4 NH + 1         TMEM allocation; one lane issues S_h = Q_h K^T of the next key tile as soon as the
//                         softmax threads have read the previous S_h.
//   warp 4 NH + 2         one lane issues O_h += P_h V of a tile once its P is complete.  Because P does not
//                         overlay S, the score product of tile j + 1 does not wait for the softmax of tile j and
//                         the PV product is off the softmax's critical path.
//   warp 4 NH + 3         idle (it completes the warpgroup that gives its registers away).
// Registers: the kernel starts with the launch-bound count for every thread; the last warpgroup then releases
// all but 56 per thread (setmaxnreg.dec) and the softmax warpgroups take them (setmaxnreg.inc).
// MMA issue: four K = 16 steps per instruction sequence with immediate offsets (mma_*_x4).  Measured on B200,
// back to back: 65 cycles per step at N = 128 (64 are pure math), 50 at N <= 64, for A in shared memory or in
// TMEM alike; a tcgen05.commit between groups of four to eight steps adds 100 to 150 cycles of tensor-pipe time.
// TMEM columns: S_h [128 h, +128); O_h [128 NH + 64 h, +64); P_h [192 NH + 64 h, +64).
// Every wait on an mbarrier is bounded (2^32 cycles); on expiry the CTA raises the plan's status word, drains its
// copies, frees its TMEM and returns.  The element mask, the tile lists and CFG sharing (second store at batch row
// b + B) are those of the plan and of the other forward kernels (paper Sections 2 and 3).
#include <cstring>
#include <mutex>

#include "litevar_tc_ptx.h"

namespace litevar {

using namespace tc;

namespace {

constexpr float kRescaleThreshold = 8.f;  // log2 units: the reference maximum moves when a tile exceeds it by more

template <int NH>
struct WsCfg {
  static constexpr int kStages = NH == 2 ? 4 : 2;
  static constexpr int kThreads = 128 * NH + 128;
  static constexpr uint32_t kTmemCols = NH == 2 ? 512 : 256;
  static constexpr int kMinCtas = NH == 2 ? 1 : 2;
  static constexpr uint32_t kColO = 128 * NH;
  static constexpr uint32_t kColP = 192 * NH;
};

template <int NH>
struct WsShared {
  static constexpr int kStages = WsCfg<NH>::kStages;
  alignas(1024) uint8_t q[NH][kTileBytes];
  alignas(1024) uint8_t k[kStages][kTileBytes];
  alignas(1024) uint8_t v[kStages][kTileBytes];
  alignas(8) uint64_t q_full;
  uint64_t k_full[kStages], k_free[kStages], v_full[kStages], v_free[kStages];
  uint64_t s_full[2], s_read[2], p_full[2], pv_done[2];
  uint32_t tmem_base;
  int abort_flag;
};

// Instruction descriptors (kind::f16): D fp32, A/B bf16, M = 128; see the field list in the other kernel.
constexpr uint32_t kIdescS = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBlockN >> 3) << 17) |
                             ((uint32_t)(kBlockM >> 4) << 24);
constexpr uint32_t kIdescO = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(kHeadDim >> 3) << 17) |
                             ((uint32_t)(kBlockM >> 4) << 24);

// 2^x for x <= 8 on the FMA pipe: x = n + f with n = round(x) and f in [-1/2, 1/2]; 2^f by a cubic fitted to it
// (relative error 7.5e-5, far inside the bf16 rounding of P), 2^n by adding n to the exponent field.  Scores of
// dead keys (-inf) are clamped to 2^-125.
__device__ __forceinline__ float2 exp2_fma2(float2 x) {
  x.x = fmaxf(x.x, -125.f);
  x.y = fmaxf(x.y, -125.f);
  const float2 t = __fadd2_rn(x, make_float2(12582912.f, 12582912.f));  // the integer part in the low mantissa bits
  const float2 n = __fadd2_rn(t, make_float2(-12582912.f, -12582912.f));
  const float2 f = __fadd2_rn(x, make_float2(-n.x, -n.y));
  float2 y = __ffma2_rn(make_float2(0.05517153441905975f, 0.05517153441905975f), f,
                        make_float2(0.2426111102104187f, 0.2426111102104187f));
  y = __ffma2_rn(y, f, make_float2(0.6932610273361206f, 0.6932610273361206f));
  y = __ffma2_rn(y, f, make_float2(0.9999280571937561f, 0.9999280571937561f));
  return make_float2(__uint_as_float(__float_as_uint(y.x) + (__float_as_uint(t.x) << 23)),
                     __uint_as_float(__float_as_uint(y.y) + (__float_as_uint(t.y) << 23)));
}

// acc += the two bf16 halves of a packed pair: fp32 additions that take a bf16 operand as it is (no unpacking)
__device__ __forceinline__ void add_bf16_pair(float2& acc, uint32_t packed) {
  asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tadd.rn.f32.bf16 %0, lo, %0;\n\tadd.rn.f32.bf16 %1, hi, %1;\n\t}"
      : "+f"(acc.x), "+f"(acc.y)
      : "r"(packed));
}

template <int N>
__device__ __forceinline__ void reg_dec() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void reg_inc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}

template <int NH>
__global__ void __launch_bounds__(WsCfg<NH>::kThreads, WsCfg<NH>::kMinCtas)
fwd_ws_kernel(const __grid_constant__ TensorMaps tm, const __grid_constant__ FwdParams p, int n_q_tiles) {
  using C = WsCfg<NH>;
  constexpr int kStages = C::kStages;
  extern __shared__ uint8_t smem_raw[];
  WsShared<NH>& sm = *reinterpret_cast<WsShared<NH>*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int kProducerWarp = 4 * NH, kMmaWarp = 4 * NH + 1, kPvWarp = 4 * NH + 2;
  int pair_rank, unit;  // grouped launch order, see cta_work
  cta_work(p, (n_q_tiles + NH - 1) / NH, pair_rank, unit);
  const int h = unit % p.n_heads, b = unit / p.n_heads;
  const int qt0 = NH == 2 ? 2 * (p.order ? __ldg(&p.order[pair_rank]) : pair_rank) : pair_rank, qt1 = qt0 + 1;
  const bool has1 = NH == 2 && qt1 < n_q_tiles;
  volatile int* abort_flag = &sm.abort_flag;

  if (threadIdx.x == kProducerWarp * 32) {
    mbar_init(&sm.q_full, 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sm.k_full[s], 1);
      mbar_init(&sm.k_free[s], 1);
      mbar_init(&sm.v_full[s], 1);
      mbar_init(&sm.v_free[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sm.s_full[i], 1);
      mbar_init(&sm.s_read[i], 4);
      mbar_init(&sm.p_full[i], 4);
      mbar_init(&sm.pv_done[i], 1);
    }
    sm.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  // the next kernel of the stream may start its set-up while this grid drains; this grid's set-up ran while the
  // previous one drained.  Nothing an earlier kernel wrote is read before the wait below.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  __syncthreads();
  if (threadIdx.x == kProducerWarp * 32) {  // Q of every half: needs nothing from the plan
    asm volatile("griddepcontrol.wait;" ::: "memory");
    mbar_expect_tx(&sm.q_full, has1 ? 2 * kTileBytes : kTileBytes);
    load_q_tile(sm.q[0], tm, p, qt0, h, b, &sm.q_full);
    if (has1) load_q_tile(sm.q[NH - 1], tm, p, qt1, h, b, &sm.q_full);
    if (p.first_tile_zero) {  // key tile 0 (cache rows [0,128), raster) heads every list: no look-up needed
      mbar_expect_tx(&sm.k_full[0], kTileBytes);
      tma_load_4d(sm.k[0], &tm.kr, 0, 0, h, b, &sm.k_full[0]);
      mbar_expect_tx(&sm.v_full[0], kTileBytes);
      tma_load_4d(sm.v[0], &tm.vr, 0, 0, h, b, &sm.v_full[0]);
    }
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                 "r"(C::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  const SetDesc sd = p.head_to_set ? p.sets[p.head_to_set[h]] : p.set0;
  const int beg0 = __ldg(&sd.row_ptr[qt0]), end0 = __ldg(&sd.row_ptr[qt0 + 1]);
  const int beg1 = end0, end1 = has1 ? __ldg(&sd.row_ptr[qt1 + 1]) : end0;
  tc_fence_before();
  __syncthreads();  // TMEM address
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp >= 4 * NH) {
    reg_dec<56>();
    if (warp == kProducerWarp && lane == 0 && end1 <= beg0) {
      // nothing listed for this CTA: only the Q copies are in flight; wait for them (bounded) before leaving
      const unsigned long long ts = global_ns();
      while (!mbar_try(&sm.q_full, 0u))
        if (global_ns() - ts > kWaitLimitNs) break;
    } else if (warp == kProducerWarp && lane == 0) {
      // ---------------------------------------------------------------- TMA producer
      UnionWalk pw;
      pw.init(sd.pairs, beg0, end0, beg1, end1);
      int issued = 0;
      if (p.first_tile_zero) {  // item 0 is already on its way
        bool l0, l1;
        (void)pw.next(l0, l1);
        issued = 1;
      }
      for (int i = issued; pw.has(); ++i) {
        bool l0, l1;
        const int kt = pw.next(l0, l1);
        const int s = i % kStages, n = i / kStages;
        if (n > 0 && !mbar_wait_inl(&sm.k_free[s], (uint32_t)((n - 1) & 1), abort_flag, p.status)) break;
        mbar_expect_tx(&sm.k_full[s], kTileBytes);
        load_kv_tile(sm.k[s], &tm.kr, tm.k2, p, kt, h, b, &sm.k_full[s]);
        if (n > 0 && !mbar_wait_inl(&sm.v_free[s], (uint32_t)((n - 1) & 1), abort_flag, p.status)) {
          const unsigned long long ts = global_ns();  // the K copy just issued is still in flight
          while (!mbar_try(&sm.k_full[s], (uint32_t)(n & 1)))
            if (global_ns() - ts > kWaitLimitNs) break;
          break;
        }
        mbar_expect_tx(&sm.v_full[s], kTileBytes);
        load_kv_tile(sm.v[s], &tm.vr, tm.v2, p, kt, h, b, &sm.v_full[s]);
        issued = i + 1;
      }
      if (*abort_flag) {  // wait (bounded) for copies still in flight before the CTA may exit
        const unsigned long long ts = global_ns();
        while (!mbar_try(&sm.q_full, 0u))
          if (global_ns() - ts > kWaitLimitNs) break;
        for (int i = issued > kStages ? issued - kStages : 0; i < issued; ++i) {
          const int s = i % kStages, n = i / kStages;
          while (!(mbar_try(&sm.k_full[s], (uint32_t)(n & 1)) && mbar_try(&sm.v_full[s], (uint32_t)(n & 1))))
            if (global_ns() - ts > 2 * kWaitLimitNs) break;
        }
      }
    } else if (warp == kMmaWarp && lane == 0 && end1 > beg0) {
      // ---------------------------------------------------------------- issuer of the score products
      const uint64_t q_desc[2] = {make_desc(smem_u32(sm.q[0])), make_desc(smem_u32(sm.q[NH - 1]))};
      const uint64_t k_desc0 = make_desc(smem_u32(sm.k[0]));
      UnionWalk w;
      w.init(sd.pairs, beg0, end0, beg1, end1);
      bool ok = mbar_wait_inl(&sm.q_full, 0u, abort_flag, p.status);
      int n_s[2] = {0, 0};  // products issued so far per half
      for (int i = 0; ok && w.has(); ++i) {
        bool live[2] = {false, false};
        const int s = i % kStages;
        (void)w.next(live[0], live[1]);
        if (!(ok = mbar_wait_inl(&sm.k_full[s], (uint32_t)((i / kStages) & 1), abort_flag, p.status))) break;
        tc_fence_after();
        const uint64_t k_desc = k_desc0 + (uint64_t)((kTileBytes >> 4) * s);
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          if (!live[hh]) continue;
          if (n_s[hh] > 0) {  // the softmax threads have read the previous S_hh
            if (!(ok = mbar_wait_inl(&sm.s_read[hh], (uint32_t)((n_s[hh] - 1) & 1), abort_flag, p.status))) break;
            tc_fence_after();
          }
          // 16 bf16 = 32 B per step inside the swizzle rows of Q and K
          mma_ss_x4<2, 2>(tmem + 128 * hh, q_desc[hh], k_desc, kIdescS, 0u);
          mma_commit(&sm.s_full[hh]);
          ++n_s[hh];
        }
        if (!ok) break;
        mma_commit(&sm.k_free[s]);
      }
    } else if (warp == kPvWarp && lane == 0 && end1 > beg0) {
      // ---------------------------------------------------------------- issuer of the PV products
      const uint64_t v_desc0 = make_desc(smem_u32(sm.v[0]));
      UnionWalk w;
      w.init(sd.pairs, beg0, end0, beg1, end1);
      bool ok = true;
      int n_pv[2] = {0, 0};
      for (int i = 0; ok && w.has(); ++i) {
        bool live[2] = {false, false};
        const int s = i % kStages;
        (void)w.next(live[0], live[1]);
        const uint64_t v_desc = v_desc0 + (uint64_t)((kTileBytes >> 4) * s);
        bool v_ready = false;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          if (!live[hh]) continue;
          if (!(ok = mbar_wait_inl(&sm.p_full[hh], (uint32_t)(n_pv[hh] & 1), abort_flag, p.status))) break;
          if (!v_ready) {
            if (!(ok = mbar_wait_inl(&sm.v_full[s], (uint32_t)((i / kStages) & 1), abort_flag, p.status))) break;
            v_ready = true;
          }
          tc_fence_after();
          // 16 keys per step = 16 rows of 128 B = 2048 B of V and 8 packed columns of P
          mma_ts_x4<8, (2048 >> 4)>(tmem + C::kColO + kHeadDim * hh, tmem + C::kColP + 64 * hh, v_desc, kIdescO,
                                    n_pv[hh] > 0 ? 1u : 0u);
          mma_ts_x4<8, (2048 >> 4)>(tmem + C::kColO + kHeadDim * hh, tmem + C::kColP + 64 * hh + 32,
                                    v_desc + 4 * (uint64_t)(2048 >> 4), kIdescO, 1u);
          mma_commit(&sm.pv_done[hh]);
          ++n_pv[hh];
        }
        if (!ok) break;
        mma_commit(&sm.v_free[s]);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue of one half
    if constexpr (NH == 2) reg_inc<224>(); else reg_inc<200>();
    const int hh = warp >> 2;
    const int qt = hh ? qt1 : qt0;
    const int pbeg = hh ? beg1 : beg0;
    const int n_tiles = (hh ? end1 : end0) - pbeg;
    if (n_tiles > 0) {
      const int lane_group = warp & 3;  // TMEM lanes this warp may touch: 32 * lane_group .. + 31
      const int m = lane_group * 32 + lane;
      const uint32_t tlane = tmem + ((uint32_t)(lane_group * 32) << 16);
      const uint32_t tS = tlane + 128 * hh;
      const uint32_t tO = tlane + C::kColO + kHeadDim * hh;
      const uint32_t tP = tlane + C::kColP + 64 * hh;
      bool ok = true;
      const float sc = p.sm_scale * 1.4426950408889634f;
      const float2 sc2 = make_float2(sc, sc);
      float row_max = -INFINITY;  // the score the stored probabilities refer to
      float2 l2a = make_float2(0.f, 0.f), l2b = make_float2(0.f, 0.f);  // row sum of the probabilities
      Pair pr = sd.pairs[pbeg];
      uint4 mk = make_uint4(~0u, ~0u, ~0u, ~0u);
      if (pr.mask_block >= 0) mk = __ldg(&sd.mask[(size_t)pr.mask_block * kBlockM + m]);
      for (int j = 0; ok && j < n_tiles; ++j) {
        Pair pr_next = pr;  // next pair's mask words travel while this tile is processed
        uint4 mk_next = make_uint4(~0u, ~0u, ~0u, ~0u);
        if (j + 1 < n_tiles) {
          pr_next = sd.pairs[pbeg + j + 1];
          if (pr_next.mask_block >= 0) mk_next = __ldg(&sd.mask[(size_t)pr_next.mask_block * kBlockM + m]);
        }
        const bool partial = pr.mask_block >= 0;
        // S_hh(j) complete
        if (!(ok = mbar_wait_inl(&sm.s_full[hh], (uint32_t)(j & 1), abort_flag, p.status))) break;
        tc_fence_after();
        // The tile is taken in two passes of 64 keys through ONE copy of the code (the loop below is kept rolled:
        // an unrolled 128-key body is some 30 KB of instructions, and two warps per scheduler streaming that
        // through the instruction caches ran at a third of the speed the same arithmetic reaches in a small
        // loop).  The probabilities refer to the running reference row_max, which a pass moves only when its own
        // maximum exceeds it by more than the threshold.  When the second pass moves it, the P written by the
        // first pass refers to the old reference: the tile is then simply redone (first pass without adding to
        // the row sum, which has been rescaled with the accumulator); S stays in TMEM until the tile is finished.
        bool pv_seen = j == 0;   // PV product of the previous tile complete: its P block is free, O_hh at rest
        bool redo = false;
#pragma unroll 1
        for (int hf = 0; hf < 2; ++hf) {
          const uint32_t w0 = hf ? mk.z : mk.x, w1 = hf ? mk.w : mk.y;
          // keys without a live key for any row of the warp are skipped (uniform over the warp)
          const bool live_h = !partial || __any_sync(0xffffffffu, (w0 | w1) != 0u);
          uint32_t pk[32];
          if (live_h) {
            uint32_t r[64];
            tmem_ld32(tS + 64 * hf, r);
            tmem_ld32(tS + 64 * hf + 32, r + 32);
            tmem_wait_ld();
            if (partial) {  // dead scores of a partially live pair become -inf
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                if (!((w0 >> e) & 1u)) r[e] = 0xff800000u;
                if (!((w1 >> e) & 1u)) r[32 + e] = 0xff800000u;
              }
            }
            if (!redo) {
              float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
              for (int e = 0; e < 64; e += 8) {
#pragma unroll
                for (int u = 0; u < 4; ++u)
                  mx[u] = max3(mx[u], __uint_as_float(r[e + 2 * u]), __uint_as_float(r[e + 2 * u + 1]));
              }
              const float pass_max = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
              // false for pass_max = -inf (no live key in this row), true for row_max = -inf (first live key)
              const bool moved = (pass_max - row_max) * sc > kRescaleThreshold;
              if (__any_sync(0xffffffffu, moved)) {
                float alpha = 1.f;
                if (moved) {
                  if (row_max != -INFINITY) alpha = fast_exp2((row_max - pass_max) * sc);
                  row_max = pass_max;
                }
                if (__any_sync(0xffffffffu, alpha != 1.f)) {  // accumulator and row sum follow the reference
                  if (!pv_seen) {
                    if (!(ok = mbar_wait_inl(&sm.pv_done[hh], (uint32_t)((j - 1) & 1), abort_flag, p.status))) break;
                    tc_fence_after();
                    pv_seen = true;
                  }
                  if (j > 0) {
#pragma unroll 1
                    for (int c = 0; c < kHeadDim / 16; ++c) {
                      uint32_t o[16];
                      tmem_ld16(tO + 16 * c, o);
                      tmem_wait_ld();
#pragma unroll
                      for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                      tmem_st16(tO + 16 * c, o);
                    }
                  }
                  l2a.x *= alpha; l2a.y *= alpha; l2b.x *= alpha; l2b.y *= alpha;
                  if (hf == 1) {  // the first pass wrote P against the old reference: redo the tile
                    redo = true;
                    hf = -1;
                    continue;
                  }
                }
              }
            }
            if (hf == 1) {  // every score of the tile has been read and no redo is pending: release the S block
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(&sm.s_read[hh]);
            }
            // probabilities against the reference: scale and shift (packed FMAs), 2^x, row sum, bf16
            const float msc = row_max == -INFINITY ? 0.f : row_max * sc;
            const float2 nm2 = make_float2(-msc, -msc);
            const bool add_sum = !(redo && hf == 0);
#pragma unroll
            for (int e = 0; e < 64; e += 4) {
              const float2 xa = __ffma2_rn(make_float2(__uint_as_float(r[e + 0]), __uint_as_float(r[e + 1])), sc2, nm2);
              const float2 xb = __ffma2_rn(make_float2(__uint_as_float(r[e + 2]), __uint_as_float(r[e + 3])), sc2, nm2);
              const float2 pa = make_float2(fast_exp2(xa.x), fast_exp2(xa.y));
              // every fourth pair on the FMA pipe: the exponential pipe (16 per clock and SM) is what a pass waits for
              const float2 pb = (e & 4) ? exp2_fma2(xb) : make_float2(fast_exp2(xb.x), fast_exp2(xb.y));
              // the row sum adds the probabilities as the PV product sees them (rounded to bf16): numerator and
              // denominator of a row then agree, and a row with one dominant key reproduces that key's V exactly
              const uint32_t ka = pack_bf16(pa.x, pa.y), kb = pack_bf16(pb.x, pb.y);
              if (add_sum) {
                add_bf16_pair(l2a, ka);
                add_bf16_pair(l2b, kb);
              }
              pk[(e >> 1) + 0] = ka;
              pk[(e >> 1) + 1] = kb;
            }
          } else {
            if (hf == 1) {
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(&sm.s_read[hh]);
            }
#pragma unroll
            for (int e = 0; e < 32; ++e) pk[e] = 0u;
          }
          if (!pv_seen) {
            if (!(ok = mbar_wait_inl(&sm.pv_done[hh], (uint32_t)((j - 1) & 1), abort_flag, p.status))) break;
            tc_fence_after();
            pv_seen = true;
          }
          tmem_st32(tP + 32 * hf, pk);
        }
        if (!ok) break;
        tmem_wait_st();  // P and, where it was rescaled, the accumulator
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.p_full[hh]);
        pr = pr_next;
        mk = mk_next;
      }
      // the last PV product of this half (all earlier ones are complete by issue order)
      if (ok && (ok = mbar_wait_inl(&sm.pv_done[hh], (uint32_t)((n_tiles - 1) & 1), abort_flag, p.status))) {
        tc_fence_after();
        uint32_t r[64];
        tmem_ld32(tO, r);
        tmem_ld32(tO + 32, r + 32);
        tmem_wait_ld();
        const float inv = 1.f / ((l2a.x + l2a.y) + (l2b.x + l2b.y));
        TileGeom g = TileGeom{-1, qt * kBlockM, 0, 0};
        if (p.q_geom != nullptr) g = p.q_geom[qt];
        int q;  // this slot's token (-1: padding slot)
        if (g.scale < 0) {
          q = g.a + m;
        } else {
          const int qr = g.a + m / kPatchCols, qc = g.b + m % kPatchCols;
          q = (qr < p.s_k && qc < p.s_k) ? qr * p.s_k + qc : -1;
        }
        if (q >= 0 && q < p.n_k) {
          uint16_t* dst = p.out + (int64_t)b * p.o_sb + (int64_t)h * p.o_sh + (int64_t)q * p.o_st;
#pragma unroll
          for (int e = 0; e < 64; e += 8) {
            uint4 o4;
            o4.x = pack_bf16(__uint_as_float(r[e + 0]) * inv, __uint_as_float(r[e + 1]) * inv);
            o4.y = pack_bf16(__uint_as_float(r[e + 2]) * inv, __uint_as_float(r[e + 3]) * inv);
            o4.z = pack_bf16(__uint_as_float(r[e + 4]) * inv, __uint_as_float(r[e + 5]) * inv);
            o4.w = pack_bf16(__uint_as_float(r[e + 6]) * inv, __uint_as_float(r[e + 7]) * inv);
            *reinterpret_cast<uint4*>(dst + e) = o4;
            if (p.share_offset > 0) *reinterpret_cast<uint4*>(dst + (int64_t)p.share_offset * p.o_sb + e) = o4;
          }
        }
      }
    }
  }

  // ---------------------------------------------------------------------- teardown (all paths)
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(C::kTmemCols) : "memory");
  }
}

template <int NH>
litevar_status_t launch_ws_variant(const TensorMaps& tm, const FwdParams& p, int n_q_tiles, cudaStream_t stream) {
  static std::once_flag attr_once;
  static cudaError_t attr_err = cudaSuccess;
  constexpr int smem_bytes = (int)sizeof(WsShared<NH>) + 1024;
  std::call_once(attr_once, [] {
    attr_err = cudaFuncSetAttribute(fwd_ws_kernel<NH>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  });
  if (attr_err != cudaSuccess) return LITEVAR_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((n_q_tiles + NH - 1) / NH) * (unsigned)p.n_heads * (unsigned)p.batch_computed);
  cfg.blockDim = dim3(WsCfg<NH>::kThreads);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = p.overlap_launch ? 1 : 0;
  if (cudaLaunchKernelEx(&cfg, fwd_ws_kernel<NH>, tm, p, n_q_tiles) != cudaSuccess) {
    (void)cudaGetLastError();
    return LITEVAR_ERR_CUDA;
  }
  return LITEVAR_OK;
}

}  // namespace

litevar_status_t launch_forward_ws(const FwdParams& p, int n_q_tiles, cudaStream_t stream) {
  TensorMaps tm;
  if (!encode_tensor_maps(p, &tm)) return LITEVAR_ERR_INVALID_ARG;
  // One query tile per CTA, two CTAs per SM: measured on B200 against the two-tile build of the same kernel (one
  // CTA per SM, K/V staged once for both tiles) it is 2 % faster on the full-mask 2K step and 4 % faster on the
  // windowed one, where the union of two tiles' lists also executes pairs that only one of them lists.  Two
  // independent CTAs drift apart, so that one's loads, masks and maxima fall under the other's exponentials.
  return launch_ws_variant<1>(tm, p, n_q_tiles, stream);
}

}  // namespace litevar
