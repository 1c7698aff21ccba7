// Tensor-core forward kernel for sm_100a: TMA-staged bf16 tiles, tcgen05 MMAs with TMEM
// accumulators, fp32 online softmax, element mask from the plan's bit blocks.
//
// One CTA handles two adjacent query tiles ("halves", 128 queries each) of one (head, batch row) and
// walks the union of their live key-tile lists in plan order, so every K/V tile is staged once for
// both halves.  640 threads:
//   warp 0       TMA producer (one lane): Q of both halves, then K and V of every listed key tile into
//                two rings of kStages tiles
//   warp 1       TMEM allocation; one lane issues, per half h, O_h += P_h V (previous tile) and then
//                S_h = Q_h K^T (next tile); the two halves alternate, so the tensor pipe works for one
//                half while the other is in its softmax
//   warps 4..11  softmax of half 0, warps 12..19 softmax of half 1.  Two threads share a query row
//                (TMEM lane): warps 4..7 / 12..15 take the first 64 keys of the tile, warps 8..11 /
//                16..19 the last 64.  Pass 1 over 16-key chunks: element mask (mixed chunks only, written
//                back to TMEM) and the row max of the thread's keys; the two partial maxima meet through
//                tagged shared-memory words that the partner polls.  The row's reference max moves only
//                when the tile exceeds it by more than 2^8; only then is the accumulator rescaled.  Pass 2:
//                exponentials against the reference, P as packed bf16 written over the first 32 of the
//                thread's own 64 S columns and handed to the PV product in two parts.  Chunks without a
//                live key for the whole warp are skipped.  The epilogue passes the rows through a per-warp
//                shared-memory slice so that four lanes store one row's 64 contiguous bytes.
// Launch: 1-D grid, query-tile pairs heaviest first; programmatic stream serialization lets the set-up of a
// call overlap the drain of the previous kernel; when every list starts with key tile 0 its copies start
// before any plan look-up.  A small build (one query tile, two stages, 384 threads, 256 TMEM columns, two
// CTAs per SM) serves steps with a single query tile or short lists.
// Row sums come from the tensor pipe: the B operand of the PV product is V (64 columns) followed by a
// block of ones (16 columns), so accumulator column 64 holds sum_t P[q,t] of the very bf16 weights the
// output uses; no per-element add is issued.
// TMEM columns: S_0 [0,128)  S_1 [128,256)  O_0 [256,336)  O_1 [336,416); P_h for keys [0,64) lies in
// S_h columns [0,32), for keys [64,128) in S_h columns [64,96).
//
// Every wait on an mbarrier or on a partner thread is bounded: when one runs out the CTA raises the plan's status
// word, drains its outstanding copies, frees its TMEM and returns.  (The TMEM allocation itself blocks while
// other CTAs on the SM hold the columns; every CTA of this library releases them before it exits.)
#include <cstring>
#include <mutex>

#include "litevar_tc_ptx.h"

namespace litevar {

using namespace tc;

namespace {

constexpr uint32_t kColS = 0;                // S_h at 128 h; O_h behind the S blocks; P_h overlays S_h
constexpr int kOutCols = kHeadDim + 16;      // V columns + the ones block (row sums)
constexpr float kRescaleThreshold = 8.f;  // log2 units
constexpr uint32_t kSlotSpinLimit = 1u << 26;  // polls of a shared-memory word before a softmax thread gives up

// Two builds of the kernel.  Full: two query tiles per CTA, four K/V stages, 640 threads, all 512 TMEM
// columns, one CTA per SM.  Lite (steps with a single query tile): one query tile, two stages, 384
// threads, 256 TMEM columns, small enough for two CTAs per SM, so that consecutive calls overlap on an SM.
template <int NH>
struct Cfg {
  static constexpr int kHalves = NH;
  static constexpr int kStages = NH == 2 ? 4 : 2;
  static constexpr int kThreads = 128 + 256 * NH;
  static constexpr uint32_t kTmemCols = 256 * NH;
  static constexpr int kMinCtas = NH == 2 ? 1 : 2;
  // 8-bit cache build: threads that widen codes: warps 0, 2 and 3, so that three of the four schedulers share the
  // work; the copy-issuing lane then sits in warp 1 beside the MMA lane.  Measured slower: the issuer inside warp 0
  // (its waits stall the 31 lanes beside it), conversion in the spare lanes of warp 1 (it delays the MMA lane), and
  // a conversion warp behind the softmax warps (21 warps are allocated as 24, which caps every thread at 80
  // registers and spills the softmax).
  static constexpr int kConvThreads = 96;
};

// 8-bit cache build: the codes of a tile (128 rows of 64 bytes, as the tensor-map copy delivers them, no swizzle)
// land in the upper half of the bf16 stage they are widened into; only the rows' scales and zero points need
// storage of their own (empty in the bf16 build).
constexpr int kCodeTileBytes = kBlockN * kHeadDim;
template <bool KV8>
struct CodeStage {};
template <>
struct CodeStage<true> {
  float sz[2][2][2][kBlockN];  // [tile parity][K, V][scale, shifted zero point][row]
};

template <int NH, bool KV8>
struct SharedStorage : CodeStage<KV8> {
  static constexpr int kStages = Cfg<NH>::kStages;
  alignas(1024) uint8_t q[NH][kTileBytes];
  alignas(1024) uint8_t k[kStages][kTileBytes];
  alignas(1024) uint8_t v[kStages][kTileBytes];
  alignas(1024) uint8_t ones[kTileBytes];  // bf16 1.0 everywhere: second N block of the PV product's B operand
  alignas(8) uint64_t q_full;
  uint64_t k_full[kStages], k_free[kStages], v_full[kStages], v_free[kStages];
  uint64_t k_codes[kStages], v_codes[kStages];  // 8-bit build: the codes of a stage have landed
  uint64_t s_full[2], p_full[2][2], o_full[2];  // p_full[h][part]: P of the first / last two chunks of each thread
  unsigned long long xslot[2][2][2][kBlockM];  // [tile parity][half][key half][row]: {tile number + 1, partial row max}
  uint32_t tmem_base;
  int abort_flag;
};

// Instruction descriptors (kind::f16): D fp32, A/B bf16, M = 128.
//   bits 4-5 D format (1 = f32), 7-9 A format (1 = bf16), 10-12 B format (1 = bf16),
//   bit 15 A major (0 = K), bit 16 B major (0 = K, 1 = MN), bits 17-22 N >> 3, bits 24-28 M >> 4.
constexpr uint32_t kIdescQK = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBlockN >> 3) << 17) |
                              ((uint32_t)(kBlockM >> 4) << 24);
constexpr uint32_t kIdescPV = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) |
                              ((uint32_t)(kOutCols >> 3) << 17) | ((uint32_t)(kBlockM >> 4) << 24);

// One tile of codes, already in registers (thread t of NT holds the 16-code chunks t, t + NT, ... of the 128 x 4
// chunks of a tile) -> bf16 rows in the 128-byte swizzle the tensor-map copies of the bf16 path produce (16-byte
// chunk c of row m at position c ^ (m & 7)).  Paper Section 4 (8-bit Q/K/V): a row enters the attention as
// code * s + z, rounded to bf16.
// The arithmetic is widen_codes16's (one fused multiply-add per pair on a shifted zero point).
// Consecutive threads write neighbouring chunks of two rows: no bank conflicts.
template <int NT>
__device__ __forceinline__ void widen_code_tile(const uint4 (&q)[(4 * kBlockN + NT - 1) / NT], uint8_t* tile,
                                                const float* scale, const float* shifted_zero, int t) {
#pragma unroll
  for (int it = 0; it < (4 * kBlockN + NT - 1) / NT; ++it) {
    const int id = t + NT * it;
    if ((4 * kBlockN) % NT != 0 && id >= 4 * kBlockN) break;
    const int m = id >> 2, c = id & 3;
    uint4 lo, hi;
    widen_codes16(q[it], scale[m], shifted_zero[m], lo, hi);
    uint8_t* row = tile + m * 128;
    *reinterpret_cast<uint4*>(row + (((2 * c) ^ (m & 7)) << 4)) = lo;
    *reinterpret_cast<uint4*>(row + (((2 * c + 1) ^ (m & 7)) << 4)) = hi;
  }
}

// Barrier of the NT conversion threads that also tells whether any of them gave up a wait, so that all take the
// same way out.
template <int NT>
__device__ __forceinline__ bool converters_sync(bool ok) {
  uint32_t any_failed;
  asm volatile(
      "{\n\t.reg .pred pin, pout;\n\tsetp.eq.u32 pin, %1, 0;\n\t"
      "bar.red.or.pred pout, 2, %2, pin;\n\tselp.u32 %0, 1, 0, pout;\n\t}"
      : "=r"(any_failed)
      : "r"((uint32_t)ok), "n"(NT)
      : "memory");
  return any_failed == 0u;
}

// The conversion warps of the 8-bit build.  The producer lane's tensor-map copies put the codes of a K (V) tile into
// the upper half of the stage; the conversion threads take them into registers, meet at a barrier (nobody reads the codes any
// more) and write the widened rows over the whole stage.  The rows' scales and zero points come by plain loads one
// tile ahead (rows past L_k: 0 and 0; their codes arrive as zeros).
template <int NH>
__device__ __forceinline__ void convert_code_tiles(SharedStorage<NH, true>& sm, const FwdParams& p, const SetDesc& sd,
                                                   int beg0, int end0, int beg1, int end1, int h, int b,
                                                   volatile int* abort_flag) {
  constexpr int kStages = Cfg<NH>::kStages;
  constexpr int NT = Cfg<NH>::kConvThreads;
  constexpr int kChunks = (4 * kBlockN + NT - 1) / NT;
  const int t = threadIdx.x < 32 ? (int)threadIdx.x : (int)threadIdx.x - 32;  // warp 0, then warps 2 and 3
  // the scales and zero points may come from the kernel just before this one in the stream: every thread that reads
  // them waits for it
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int64_t zoff = (int64_t)b * p.z_sb + (int64_t)h * p.z_sh;
  float rk[2][2], rv[2][2];  // rows t and t + NT of the tile after the one being converted
  auto fetch_rows = [&](int kt) {
    const int row0 = p.key_geom ? p.key_geom[kt].a : kt * kBlockN;  // raster tiles only
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      if (kBlockN % NT != 0 && t + NT * r >= kBlockN) break;
      const int row = row0 + t + NT * r;
      const bool valid = row < p.L_k;
      const int64_t at = zoff + (valid ? row : 0);
      rk[r][0] = valid ? __ldg(p.k_scale + at) : 0.f;
      rk[r][1] = valid ? __ldg(p.k_zero + at) : 0.f;
      rv[r][0] = valid ? __ldg(p.v_scale + at) : 0.f;
      rv[r][1] = valid ? __ldg(p.v_zero + at) : 0.f;
    }
  };
  auto take_codes = [&](const uint8_t* stage, uint4 (&q)[kChunks]) {
#pragma unroll
    for (int it = 0; it < kChunks; ++it)
      if ((4 * kBlockN) % NT == 0 || t + NT * it < 4 * kBlockN) q[it] = *reinterpret_cast<const uint4*>(stage + kCodeTileBytes + (t + NT * it) * 16);
  };
  UnionWalk row_walk, walk;
  walk.init(sd.pairs, beg0, end0, beg1, end1);
  row_walk = walk;
  bool l0, l1;
  fetch_rows(row_walk.next(l0, l1));  // the list is not empty
  for (int i = 0; walk.has(); ++i) {
    (void)walk.next(l0, l1);
    const int s = i % kStages, par = i & 1;
    const uint32_t ph = (uint32_t)((i / kStages) & 1);
    uint4 q[kChunks];
    bool ok = mbar_wait(&sm.k_codes[s], ph, abort_flag, p.status);
    if (ok) take_codes(sm.k[s], q);
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      if (kBlockN % NT != 0 && t + NT * r >= kBlockN) break;
      sm.sz[par][0][0][t + NT * r] = rk[r][0];
      sm.sz[par][0][1][t + NT * r] = shifted_zero_point(rk[r][1], rk[r][0]);
      sm.sz[par][1][0][t + NT * r] = rv[r][0];
      sm.sz[par][1][1][t + NT * r] = shifted_zero_point(rv[r][1], rv[r][0]);
    }
    if (!converters_sync<NT>(ok)) break;
    if (row_walk.has()) fetch_rows(row_walk.next(l0, l1));
    widen_code_tile<NT>(q, sm.k[s], sm.sz[par][0][0], sm.sz[par][0][1], t);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> the tensor pipe's reads
    mbar_arrive(&sm.k_full[s]);
    ok = mbar_wait(&sm.v_codes[s], ph, abort_flag, p.status);
    if (ok) take_codes(sm.v[s], q);
    if (!converters_sync<NT>(ok)) break;
    widen_code_tile<NT>(q, sm.v[s], sm.sz[par][1][0], sm.sz[par][1][1], t);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    mbar_arrive(&sm.v_full[s]);
  }
}

template <int NH, bool KV8>
__global__ void __launch_bounds__(Cfg<NH>::kThreads, Cfg<NH>::kMinCtas)
fwd_tc_kernel(const __grid_constant__ TensorMaps tm, const __grid_constant__ FwdParams p, int n_q_tiles) {
  constexpr int kStages = Cfg<NH>::kStages;
  constexpr int kThreads = Cfg<NH>::kThreads;
  constexpr uint32_t kTmemCols = Cfg<NH>::kTmemCols;
  extern __shared__ uint8_t smem_raw[];
  constexpr uint32_t kColO = 128 * NH;
  SharedStorage<NH, KV8>& sm = *reinterpret_cast<SharedStorage<NH, KV8>*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // 1-D grid, heaviest query-tile pairs first: all (head, batch row) units of a pair are neighbours
  int pair_rank, unit;  // grouped launch order, see cta_work
  cta_work(p, (n_q_tiles + NH - 1) / NH, pair_rank, unit);
  const int h = unit % p.n_heads, b = unit / p.n_heads;
  // the launch order lists query-tile PAIRS; the one-tile build takes the tiles in natural order
  const int qt0 = NH == 2 ? 2 * (p.order ? __ldg(&p.order[pair_rank]) : pair_rank) : pair_rank, qt1 = qt0 + 1;
  const bool has1 = NH == 2 && qt1 < n_q_tiles;
  volatile int* abort_flag = &sm.abort_flag;

  if (threadIdx.x == 0) {
    mbar_init(&sm.q_full, 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sm.k_full[s], KV8 ? Cfg<NH>::kConvThreads : 1);  // 8-bit cache: every conversion thread arrives
      mbar_init(&sm.k_free[s], 1);
      mbar_init(&sm.v_full[s], KV8 ? Cfg<NH>::kConvThreads : 1);
      mbar_init(&sm.k_codes[s], 1);
      mbar_init(&sm.v_codes[s], 1);
      mbar_init(&sm.v_free[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sm.s_full[i], 1);
      mbar_init(&sm.p_full[i][0], 8);
      mbar_init(&sm.p_full[i][1], 8);
      mbar_init(&sm.o_full[i], 1);
    }
    sm.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  // Programmatic dependent launch: the next kernel in the stream may start its own set-up while this grid
  // drains; this grid's set-up above ran while the previous one drained.  Nothing written by an earlier
  // kernel is read before the wait below (the plan is immutable, Q/K/V are read by the producer lane only).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  __syncthreads();  // barriers initialised; the producer warp goes ahead, the others finish the set-up
  if (threadIdx.x == 0) {  // Q of both halves: needs nothing from the plan
    asm volatile("griddepcontrol.wait;" ::: "memory");
    mbar_expect_tx(&sm.q_full, has1 ? 2 * kTileBytes : kTileBytes);
    load_q_tile(sm.q[0], tm, p, qt0, h, b, &sm.q_full);
    if (has1) load_q_tile(sm.q[NH - 1], tm, p, qt1, h, b, &sm.q_full);
    if (!KV8 && p.first_tile_zero) {  // key tile 0 (cache rows [0,128), raster) heads every list: no look-up needed
      mbar_expect_tx(&sm.k_full[0], kTileBytes);
      tma_load_4d(sm.k[0], &tm.kr, 0, 0, h, b, &sm.k_full[0]);
      mbar_expect_tx(&sm.v_full[0], kTileBytes);
      tma_load_4d(sm.v[0], &tm.vr, 0, 0, h, b, &sm.v_full[0]);
    }
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (warp != 0) {  // the ones block; made visible to the tensor pipe (async proxy) before the barrier below
    uint4* o4 = reinterpret_cast<uint4*>(sm.ones);
    for (int i = threadIdx.x - 32; i < (int)(kTileBytes / 16); i += kThreads - 32)
      o4[i] = make_uint4(0x3f803f80u, 0x3f803f80u, 0x3f803f80u, 0x3f803f80u);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    // the exchange words of the softmax threads start with a tag no tile uses
    unsigned long long* xs = &sm.xslot[0][0][0][0];
    for (int i = threadIdx.x - 32; i < 8 * kBlockM; i += kThreads - 32) xs[i] = 0ull;
  }
  // plan lookups (independent of the set-up above)
  const SetDesc sd = p.head_to_set ? p.sets[p.head_to_set[h]] : p.set0;
  const int beg0 = __ldg(&sd.row_ptr[qt0]), end0 = __ldg(&sd.row_ptr[qt0 + 1]);
  const int beg1 = end0, end1 = has1 ? __ldg(&sd.row_ptr[qt1 + 1]) : end0;
  tc_fence_before();
  if (warp != 0) asm volatile("bar.sync 1, %0;" ::"n"(kThreads - 32) : "memory");  // TMEM address, ones block
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp < 4) {
    if (warp == 0 && lane == 0 && end1 <= beg0) {
      // nothing listed for this CTA: only the Q copies are in flight; wait for them (bounded) before leaving
      const unsigned long long ts = global_ns();
      while (!mbar_try(&sm.q_full, 0u))
        if (global_ns() - ts > kWaitLimitNs) break;
    } else if (KV8 ? (warp == 1 && lane == 1) : (warp == 0 && lane == 0)) {
      // ---------------------------------------------------------------- TMA producer (8-bit build: in the MMA warp)
      // bf16 cache: a copy fills a stage and completes k_full / v_full.  8-bit cache: a copy brings the 8 KB of codes
      // of a tile into the upper half of the stage and completes k_codes / v_codes; the conversion warps then write
      // the stage and complete k_full / v_full.
      constexpr uint32_t kCopyBytes = KV8 ? kCodeTileBytes : kTileBytes;
      constexpr uint32_t kCopyAt = KV8 ? kCodeTileBytes : 0;
      auto k_bar = [&](int s) { return KV8 ? &sm.k_codes[s] : &sm.k_full[s]; };
      auto v_bar = [&](int s) { return KV8 ? &sm.v_codes[s] : &sm.v_full[s]; };
      UnionWalk pw;
      pw.init(sd.pairs, beg0, end0, beg1, end1);
      int issued = 0;
      if (!KV8 && p.first_tile_zero) {  // item 0 is already on its way
        bool l0, l1;
        (void)pw.next(l0, l1);
        issued = 1;
      }
      for (int i = issued; pw.has(); ++i) {
        bool l0, l1;
        const int kt = pw.next(l0, l1);
        const int s = i % kStages, n = i / kStages;
        if (n > 0 && !mbar_wait(&sm.k_free[s], (uint32_t)((n - 1) & 1), abort_flag, p.status)) break;
        mbar_expect_tx(k_bar(s), kCopyBytes);
        load_kv_tile(sm.k[s] + kCopyAt, &tm.kr, tm.k2, p, kt, h, b, k_bar(s));
        if (n > 0 && !mbar_wait(&sm.v_free[s], (uint32_t)((n - 1) & 1), abort_flag, p.status)) {
          // the K copy just issued is still in flight
          const unsigned long long ts = global_ns();
          while (!mbar_try(k_bar(s), (uint32_t)(n & 1)))
            if (global_ns() - ts > kWaitLimitNs) break;
          break;
        }
        mbar_expect_tx(v_bar(s), kCopyBytes);
        load_kv_tile(sm.v[s] + kCopyAt, &tm.vr, tm.v2, p, kt, h, b, v_bar(s));
        issued = i + 1;
      }
      if (*abort_flag) {
        // wait (bounded) for copies still in flight before the CTA may exit
        const unsigned long long ts = global_ns();
        while (!mbar_try(&sm.q_full, 0u))
          if (global_ns() - ts > kWaitLimitNs) break;
        for (int i = issued > kStages ? issued - kStages : 0; i < issued; ++i) {
          const int s = i % kStages, n = i / kStages;
          while (!(mbar_try(k_bar(s), (uint32_t)(n & 1)) && mbar_try(v_bar(s), (uint32_t)(n & 1))))
            if (global_ns() - ts > 2 * kWaitLimitNs) break;
        }
      }
    } else if (KV8 && warp != 1 && end1 > beg0) {
      // ---------------------------------------------------------------- 8-bit cache: widen the codes of each stage
      if constexpr (KV8) convert_code_tiles<NH>(sm, p, sd, beg0, end0, beg1, end1, h, b, abort_flag);
    } else if (warp == 1 && lane == 0 && end1 > beg0) {
      // ---------------------------------------------------------------- MMA issuer
      const uint64_t q_desc[2] = {make_desc(smem_u32(sm.q[0])), make_desc(smem_u32(sm.q[NH - 1]))};
      UnionWalk w;
      w.init(sd.pairs, beg0, end0, beg1, end1);
      bool ok = mbar_wait(&sm.q_full, 0u, abort_flag, p.status);
      int n_pv[2] = {0, 0};
      bool prev_live[2] = {false, false};
      int prev_stage = 0;
      uint32_t prev_phase = 0;
      for (int i = 0; ok; ++i) {
        const bool have = w.has();
        bool live[2] = {false, false};
        const int s = i % kStages;
        const uint32_t ph = (uint32_t)((i / kStages) & 1);
        uint64_t k_desc = 0;
        if (have) {
          (void)w.next(live[0], live[1]);
          if (!(ok = mbar_wait(&sm.k_full[s], ph, abort_flag, p.status))) break;
          tc_fence_after();
          k_desc = make_desc(smem_u32(sm.k[s]));
        }
        bool v_ready = false;
        const uint32_t v_addr = smem_u32(sm.v[prev_stage]);
        const uint64_t v_desc = make_desc_mn(v_addr, smem_u32(sm.ones) - v_addr);
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          if (i > 0 && prev_live[hh]) {  // O_hh += P_hh [V | 1]; P_hh sits in S_hh's columns
            // P arrives in two parts: key groups {0,1,4,5} (first two chunks of both threads of a row), then {2,3,6,7}
            if (!(ok = mbar_wait(&sm.p_full[hh][0], (uint32_t)(n_pv[hh] & 1), abort_flag, p.status))) break;
            if (!v_ready) {
              if (!(ok = mbar_wait(&sm.v_full[prev_stage], prev_phase, abort_flag, p.status))) break;
              v_ready = true;
            }
            tc_fence_after();
#pragma unroll
            for (int part = 0; part < 2; ++part) {
              if (part == 1) {
                if (!(ok = mbar_wait(&sm.p_full[hh][1], (uint32_t)(n_pv[hh] & 1), abort_flag, p.status))) break;
                tc_fence_after();
              }
              // four steps of 16 keys (16 rows of 128 B = 2048 B of V, 8 packed columns of P) in one instruction
              // sequence: key groups {0, 1, 4, 5} for the first part, {2, 3, 6, 7} for the second; the second key
              // half of P starts at S column 64
              mma_ts_x4_at<8, 64, 72, 128, 512, 640>(tmem + kColO + kOutCols * hh, tmem + kColS + 128 * hh + 16 * part,
                                                     v_desc + (uint64_t)(2 * 128) * part, kIdescPV,
                                                     (n_pv[hh] > 0 || part > 0) ? 1u : 0u);
            }
            if (!ok) break;
            mma_commit(&sm.o_full[hh]);
            ++n_pv[hh];
          }
          if (have && live[hh]) {  // S_hh = Q_hh K^T, after the PV above in issue order
            // 16 bf16 = 32 B per step inside the swizzle rows of Q and K
            mma_ss_x4<2, 2>(tmem + kColS + 128 * hh, q_desc[hh], k_desc, kIdescQK, 0u);
            mma_commit(&sm.s_full[hh]);
          }
        }
        if (!ok) break;
        if (have) mma_commit(&sm.k_free[s]);
        if (i > 0) mma_commit(&sm.v_free[prev_stage]);
        if (!have) break;
        prev_live[0] = live[0];
        prev_live[1] = live[1];
        prev_stage = s;
        prev_phase = ph;
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue of one half
    const int hh = (warp - 4) >> 3;        // query half
    const int sub = ((warp - 4) >> 2) & 1;  // key half of every tile this thread works on
    const int qt = hh ? qt1 : qt0;
    const int pbeg = hh ? beg1 : beg0;
    const int n_tiles = (hh ? end1 : end0) - pbeg;
    if (n_tiles > 0) {
      const int lane_group = warp & 3;  // TMEM lanes this warp may touch: 32*lane_group .. +31
      const int m = lane_group * 32 + lane;
      const uint32_t tlane = tmem + ((uint32_t)(lane_group * 32) << 16);
      const uint32_t tS = tlane + kColS + 128 * hh + 64 * sub;  // this thread's 64 score columns
      const uint32_t tO = tlane + kColO + kOutCols * hh;
      const float sc = p.sm_scale * 1.4426950408889634f;
      float row_max = -INFINITY;  // the score the stored probabilities refer to
      bool ok = true;
      Pair pr = sd.pairs[pbeg];
      uint2 mk = make_uint2(~0u, ~0u);
      if (pr.mask_block >= 0)
        mk = __ldg(reinterpret_cast<const uint2*>(&sd.mask[(size_t)pr.mask_block * kBlockM + m]) + sub);
      for (int j = 0; j < n_tiles; ++j) {
        // next pair's mask words travel while this tile is processed
        Pair pr_next = pr;
        uint2 mk_next = make_uint2(~0u, ~0u);
        if (j + 1 < n_tiles) {
          pr_next = sd.pairs[pbeg + j + 1];
          if (pr_next.mask_block >= 0)
            mk_next = __ldg(reinterpret_cast<const uint2*>(&sd.mask[(size_t)pr_next.mask_block * kBlockM + m]) + sub);
        }
        const bool partial = pr.mask_block >= 0;
        // per 16-key chunk, uniform over the warp: 0 = no live key (skipped), 1 = mixed, 2 = all live
        uint32_t wbits[4] = {mk.x & 0xffffu, mk.x >> 16, mk.y & 0xffffu, mk.y >> 16};
        int chunk_kind[4];
        bool any_mixed = false;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          chunk_kind[c] = 2;
          if (partial)
            chunk_kind[c] = !__any_sync(0xffffffffu, wbits[c] != 0u) ? 0
                            : (__all_sync(0xffffffffu, wbits[c] == 0xffffu) ? 2 : 1);
          any_mixed |= chunk_kind[c] == 1;
        }
        // S_hh(j) complete; in issue order this also means the PV product of tile j-1 is complete
        if (!(ok = mbar_wait(&sm.s_full[hh], (uint32_t)(j & 1), abort_flag, p.status))) break;
        tc_fence_after();
        uint32_t r[2][16];
        // ---- pass 1: mask the mixed chunks (written back) and take the max of this thread's 64 keys
        float mx0 = -INFINITY, mx1 = -INFINITY;
        tmem_ld16(tS, r[0]);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t* rc = r[c & 1];
          tmem_wait_ld();
          if (c + 1 < 4) tmem_ld16(tS + 16 * (c + 1), r[(c + 1) & 1]);
          if (chunk_kind[c] == 0) continue;
          if (chunk_kind[c] == 1) {
#pragma unroll
            for (int e = 0; e < 16; ++e)
              if (!((wbits[c] >> e) & 1u)) rc[e] = 0xff800000u;  // -inf
            tmem_st16(tS + 16 * c, rc);
          }
#pragma unroll
          for (int e = 0; e < 16; e += 4) {
            mx0 = max3(mx0, __uint_as_float(rc[e + 0]), __uint_as_float(rc[e + 1]));
            mx1 = max3(mx1, __uint_as_float(rc[e + 2]), __uint_as_float(rc[e + 3]));
          }
        }
        // the scores of the second pass start travelling while the maxima are exchanged
        if (any_mixed) tmem_wait_st();  // the masked scores are read back
        tmem_ld16(tS, r[0]);
        // the two threads of a row exchange their maxima
        float tile_max = fmaxf(mx0, mx1);
        // (one 8-byte shared-memory word per thread and tile parity, tagged with the tile number: the partner
        // polls it; it can be at most one tile ahead, so two parities suffice)
        {
          volatile unsigned long long* mine = &sm.xslot[j & 1][hh][sub][m];
          volatile unsigned long long* theirs = &sm.xslot[j & 1][hh][sub ^ 1][m];
          *mine = ((unsigned long long)(uint32_t)(j + 1) << 32) | __float_as_uint(tile_max);
          unsigned long long got = *theirs;
          for (uint32_t spin = 0; (uint32_t)(got >> 32) != (uint32_t)(j + 1); ++spin) {
            if ((spin & 1023u) == 1023u && (*abort_flag || spin > kSlotSpinLimit)) {
              *abort_flag = 1;
              atomicExch(p.status, 1);
              ok = false;
              break;
            }
            got = *theirs;
          }
          if (!__all_sync(0xffffffffu, ok)) {
            ok = false;
            break;
          }
          tile_max = fmaxf(tile_max, __uint_as_float((uint32_t)got));
        }
        // the reference max moves only when the tile exceeds it by more than the threshold
        float alpha = 1.f;
        if ((tile_max - row_max) * sc > kRescaleThreshold) {  // false for tile_max = -inf, true for row_max = -inf
          if (row_max != -INFINITY) alpha = fast_exp2((row_max - tile_max) * sc);
          row_max = tile_max;
        }
        if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
          // accumulator and row sum follow the reference: columns [0,48) here, [48,80) in the partner thread
          uint32_t o[16];
#pragma unroll
          for (int c = 0; c < 3 - sub; ++c) {
            const uint32_t col = 48 * sub + 16 * c;
            tmem_ld16(tO + col, o);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st16(tO + col, o);
          }
        }
        // ---- pass 2: probabilities against the reference; P (packed bf16) over this thread's first 32 columns
        const float msc = row_max == -INFINITY ? 0.f : row_max * sc;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t* rc = r[c & 1];
          tmem_wait_ld();
          if (c + 1 < 4) tmem_ld16(tS + 16 * (c + 1), r[(c + 1) & 1]);
          uint32_t pk[8];
          if (chunk_kind[c] != 0) {
#pragma unroll
            for (int e = 0; e < 16; e += 2) {
              const float p0 = fast_exp2(fmaf(__uint_as_float(rc[e + 0]), sc, -msc));
              const float p1 = fast_exp2(fmaf(__uint_as_float(rc[e + 1]), sc, -msc));
              pk[e >> 1] = pack_bf16(p0, p1);
            }
          } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) pk[e] = 0u;
          }
          tmem_st8(tS + 8 * c, pk);  // columns [8c, 8c+8) of this thread's 64: inside chunks already read
          if (c == 1) {  // first half of P can enter the PV product while the rest is formed
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.p_full[hh][0]);
          }
        }
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.p_full[hh][1]);
        pr = pr_next;
        mk = mk_next;
      }
      // the last PV product of this half (all earlier ones are complete by issue order)
      if (ok && (ok = mbar_wait(&sm.o_full[hh], (uint32_t)((n_tiles - 1) & 1), abort_flag, p.status))) {
        tc_fence_after();
        uint32_t l16[16];
        tmem_ld16(tO + kHeadDim, l16);  // row sum of the bf16 probabilities, from the ones block
        uint32_t r[32];
        tmem_ld32(tO + 32 * sub, r);    // output columns [32 sub, 32 sub + 32) of this thread's row
        tmem_wait_ld();
        const float inv = 1.f / __uint_as_float(l16[0]);
        // The warp's 32 rows x 64 B pass through its own 2 KB slice of the half's Q buffer (its last reader,
        // S_hh of the last tile, is done), so that four neighbouring lanes store one row's 64 contiguous
        // bytes instead of 32 lanes touching 32 different rows.  Chunk position XOR (row / 2) keeps both
        // the writes and the reads free of bank conflicts.  No other warp touches the slice.
        uint8_t* slice = sm.q[hh < NH ? hh : 0] + (((warp - 4) & 7) << 11);
#pragma unroll
        for (int e = 0; e < 32; e += 8) {
          uint4 o4;
          o4.x = pack_bf16(__uint_as_float(r[e + 0]) * inv, __uint_as_float(r[e + 1]) * inv);
          o4.y = pack_bf16(__uint_as_float(r[e + 2]) * inv, __uint_as_float(r[e + 3]) * inv);
          o4.z = pack_bf16(__uint_as_float(r[e + 4]) * inv, __uint_as_float(r[e + 5]) * inv);
          o4.w = pack_bf16(__uint_as_float(r[e + 6]) * inv, __uint_as_float(r[e + 7]) * inv);
          *reinterpret_cast<uint4*>(slice + lane * 64 + ((((e >> 3) ^ (lane >> 1)) & 3) << 4)) = o4;
        }
        __syncwarp();
        TileGeom g = TileGeom{-1, qt * kBlockM, 0, 0};
        if (p.q_geom != nullptr) g = p.q_geom[qt];
        uint16_t* obase = p.out + (int64_t)b * p.o_sb + (int64_t)h * p.o_sh + 32 * sub;
#pragma unroll
        for (int it = 0; it < 4; ++it) {
          const int rl = it * 8 + (lane >> 2), ch = lane & 3;  // row of the warp's 32, 16-byte chunk of its 64 bytes
          const int mm = lane_group * 32 + rl;                  // query slot of that row
          int q;                                                // its token (-1: padding slot)
          if (g.scale < 0) {
            q = g.a + mm;
          } else {
            const int qr = g.a + mm / kPatchCols, qc = g.b + mm % kPatchCols;
            q = (qr < p.s_k && qc < p.s_k) ? qr * p.s_k + qc : -1;
          }
          const uint4 o4 = *reinterpret_cast<const uint4*>(slice + rl * 64 + (((ch ^ (rl >> 1)) & 3) << 4));
          if (q >= 0 && q < p.n_k) {
            uint16_t* dst = obase + (int64_t)q * p.o_st + 8 * ch;
            *reinterpret_cast<uint4*>(dst) = o4;
            if (p.share_offset > 0) *reinterpret_cast<uint4*>(dst + (int64_t)p.share_offset * p.o_sb) = o4;
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
bool encode_raster(CUtensorMap* tm, const void* base, int64_t rows, int64_t heads, int64_t batch, int64_t st,
                   int64_t sh, int64_t sb) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  if (rows < 1) rows = 1;  // no raster tile will use this map
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

// Rank-4 map over a [batch, head, token, 64] tensor of 8-bit codes with byte strides (multiples of 16); box = 128
// tokens x 64 bytes, rows packed in shared memory without swizzle.  Rows past the last one read as zero.
bool encode_codes(CUtensorMap* tm, const void* base, int64_t rows, int64_t heads, int64_t batch, int64_t st,
                  int64_t sh, int64_t sb) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  if (rows < 1) rows = 1;
  if (heads == 1 && sh < kHeadDim) sh = st * rows;
  if (batch == 1 && sb < kHeadDim) sb = sh * heads;
  cuuint64_t gdim[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)rows, (cuuint64_t)heads, (cuuint64_t)batch};
  cuuint64_t gstr[3] = {(cuuint64_t)st, (cuuint64_t)sh, (cuuint64_t)sb};
  cuuint32_t box[4] = {(cuuint32_t)kHeadDim, (cuuint32_t)kBlockN, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), gdim, gstr, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Rank-5 map over the side x side grid of one scale inside a [batch, head, token, 64] tensor: dimensions
// (64, column, row, head, batch); box = 8 rows x 16 columns x 64, i.e. 128 rows of 128 B in shared memory in
// row-major patch order.  Cells outside the grid read as zero and are not written.
bool encode_patch(CUtensorMap* tm, const void* base, int64_t first_token, int64_t side, int64_t heads,
                  int64_t batch, int64_t st, int64_t sh, int64_t sb) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  if (heads == 1 && sh < kHeadDim) sh = st * side * side;
  if (batch == 1 && sb < kHeadDim) sb = sh * heads;
  const uint16_t* origin = static_cast<const uint16_t*>(base) + first_token * st;
  cuuint64_t gdim[5] = {(cuuint64_t)kHeadDim, (cuuint64_t)side, (cuuint64_t)side, (cuuint64_t)heads, (cuuint64_t)batch};
  cuuint64_t gstr[4] = {(cuuint64_t)st * 2, (cuuint64_t)(st * side) * 2, (cuuint64_t)sh * 2, (cuuint64_t)sb * 2};
  cuuint32_t box[5] = {(cuuint32_t)kHeadDim, (cuuint32_t)kPatchCols, (cuuint32_t)kPatchRows, 1, 1};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<uint16_t*>(origin), gdim, gstr, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

template <int NH, bool KV8>
litevar_status_t launch_variant(const TensorMaps& tm, const FwdParams& p, int n_q_tiles, cudaStream_t stream) {
  static std::once_flag attr_once;
  static cudaError_t attr_err = cudaSuccess;
  constexpr int smem_bytes = (int)sizeof(SharedStorage<NH, KV8>) + 1024;
  std::call_once(attr_once, [] {
    attr_err = cudaFuncSetAttribute(fwd_tc_kernel<NH, KV8>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  });
  if (attr_err != cudaSuccess) return LITEVAR_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((n_q_tiles + NH - 1) / NH) * (unsigned)p.n_heads * (unsigned)p.batch_computed);
  cfg.blockDim = dim3(Cfg<NH>::kThreads);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = p.overlap_launch ? 1 : 0;  // off when an earlier kernel of the stream writes what the set-up reads
  if (cudaLaunchKernelEx(&cfg, fwd_tc_kernel<NH, KV8>, tm, p, n_q_tiles) != cudaSuccess) {
    (void)cudaGetLastError();
    return LITEVAR_ERR_CUDA;
  }
  return LITEVAR_OK;
}

}  // namespace

bool encode_tensor_maps(const FwdParams& p, tc::TensorMaps* tmp) {
  tc::TensorMaps& tm = *tmp;
  memset(&tm, 0, sizeof(tm));
  bool ok;
  if (p.q_patch)
    ok = encode_patch(&tm.q, p.q, 0, p.s_k, p.n_heads, p.batch_computed, p.q_st, p.q_sh, p.q_sb);
  else
    ok = encode_raster(&tm.q, p.q, p.n_k, p.n_heads, p.batch_computed, p.q_st, p.q_sh, p.q_sb);
  ok = ok && encode_raster(&tm.kr, p.k, p.raster_len, p.n_heads, p.batch_computed, p.k_st, p.k_sh, p.k_sb) &&
       encode_raster(&tm.vr, p.v, p.raster_len, p.n_heads, p.batch_computed, p.v_st, p.v_sh, p.v_sb);
  for (int i = 0; ok && i < p.n_patch_scales; ++i)
    ok = encode_patch(&tm.k2[i], p.k, p.patch_off[i], p.patch_scale[i], p.n_heads, p.batch_computed, p.k_st, p.k_sh,
                      p.k_sb) &&
         encode_patch(&tm.v2[i], p.v, p.patch_off[i], p.patch_scale[i], p.n_heads, p.batch_computed, p.v_st, p.v_sh,
                      p.v_sb);
  return ok;
}

litevar_status_t launch_forward_tcgen05(const FwdParams& p, int n_q_tiles, cudaStream_t stream) {
  TensorMaps tm;
  if (!encode_tensor_maps(p, &tm)) return LITEVAR_ERR_INVALID_ARG;
  // A step with a single query tile and more CTAs than SMs runs the small build: two CTAs share an SM and
  // hide each other's set-up and drain.  With fewer CTAs than SMs sharing would only halve each CTA's SM.
  const int n_sm = current_sm_count();
  const long long units = (long long)p.n_heads * p.batch_computed;
  // ... and so does a step whose lists are short (set-up and drain weigh more than the shared K/V staging saves)
  const bool lite = (n_q_tiles == 1 && units > n_sm) ||
                    (units * n_q_tiles >= 2LL * n_sm && p.pairs_per_tile > 0 && p.pairs_per_tile <= 14);
  return lite ? launch_variant<1, false>(tm, p, n_q_tiles, stream) : launch_variant<2, false>(tm, p, n_q_tiles, stream);
}

litevar_status_t launch_forward_tcgen05_kv8(const FwdParams& p, int n_q_tiles, cudaStream_t stream) {
  TensorMaps tm;
  memset(&tm, 0, sizeof(tm));
  // the raster maps of K and V cover the code tensors here
  if (!encode_raster(&tm.q, p.q, p.n_k, p.n_heads, p.batch_computed, p.q_st, p.q_sh, p.q_sb) ||
      !encode_codes(&tm.kr, p.k8, p.L_k, p.n_heads, p.batch_computed, p.c_st, p.c_sh, p.c_sb) ||
      !encode_codes(&tm.vr, p.v8, p.L_k, p.n_heads, p.batch_computed, p.c_st, p.c_sh, p.c_sb))
    return LITEVAR_ERR_INVALID_ARG;
  const int n_sm = current_sm_count();
  const long long units = (long long)p.n_heads * p.batch_computed;
  // two query tiles per CTA wherever there are two: a widened K/V tile then serves both
  const bool lite = n_q_tiles == 1 && units > n_sm;
  return lite ? launch_variant<1, true>(tm, p, n_q_tiles, stream) : launch_variant<2, true>(tm, p, n_q_tiles, stream);
}

}  // namespace litevar
