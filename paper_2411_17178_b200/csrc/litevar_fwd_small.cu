// Forward kernel for the small steps of the schedule: one query tile, at most two raster key tiles
// and little work (n_k x L_k up to about 96 x 192: the first six or seven steps of the paper's 256px and 512px
// schedules).
//
// Such a step is a chain of latencies, not a stream of tiles: the tcgen05 kernel spends it on TMEM allocation,
// descriptor set-up and four mbarrier hand-offs around one MMA pair.  Here one CTA per (batch row, head) stages
// Q and the whole K/V prefix in shared memory with one round of 16-byte asynchronous copies, and every warp
// takes 16 query rows through S = Q K^T, the masked softmax and O = P V with warp-level mma (m16n8k16, bf16
// in, fp32 accumulate), S and P never leaving registers.  There is no wait on another thread's progress
// anywhere but one __syncthreads.
//
// Same plan, same element-mask blocks, same arithmetic contract as the tensor-core kernel (paper Section 2:
// scores of dead keys are removed before the softmax, which renormalises over the live keys; Section 3: at a
// shared step the result is stored to the conditional and the unconditional row).  P is rounded to bf16 before
// P V and the row sum adds the rounded values.
#include <cuda_runtime.h>

#include <mutex>

#include "litevar_internal.h"

namespace litevar {

namespace {

constexpr int kRowPad = 72;        // bf16 elements per staged row: 144 B keeps ldmatrix rows on distinct banks
constexpr int kSmallMaxWarps = 8;  // 16 query rows each
constexpr int kMergePad = 68;      // floats per row of a partial output handed from one warp of a pair to the other
constexpr int kMergeFloats = 16 * kMergePad + 32;  // per row group: 16 partial output rows, 16 maxima, 16 sums

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr(dst)), "l"(src) : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(smem_addr(p)));
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(smem_addr(p)));
}

// d += a (16x16, row) * b (16x8, col), bf16 operands, fp32 accumulators
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// two floats -> packed bf16 pair (round to nearest even), low half = first
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// SPLIT = 1: one warp per 16 query rows.  SPLIT = 2: two warps per 16 query rows, each taking every other
// 64-key round, merged through shared memory at the end; for launches that leave SMs to spare, where the
// chain of rounds of a single warp is what the call waits for.
template <int SPLIT, bool KV8>
__global__ void __launch_bounds__(kSmallMaxWarps * 32 * SPLIT) fwd_small_kernel(FwdParams p, SmallLists lists) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int q_rows = ((p.n_k + 15) >> 4) * 16;  // 16 per computing warp; further warps only help staging
  const int l_pad = (p.L_k + 15) & ~15;
  uint16_t* Qs = reinterpret_cast<uint16_t*>(smem_raw);  // [q_rows][kRowPad]; later the output rows
  uint16_t* Ks = Qs + q_rows * kRowPad;                   // [l_pad][kRowPad]
  uint16_t* Vs = Ks + l_pad * kRowPad;                    // [l_pad][kRowPad]
  uint32_t* Ms = reinterpret_cast<uint32_t*>(Vs + l_pad * kRowPad);  // [q_rows][8]: live bits of keys 0 .. 255
  float* Xs = reinterpret_cast<float*>(Ms + q_rows * 8);             // SPLIT 2: [q_rows / 16][kMergeFloats]

  asm volatile("griddepcontrol.launch_dependents;");
  const int h = blockIdx.x % p.n_heads, b = blockIdx.x / p.n_heads;

  // ---- live bits per query row: plan data, complete before any forward was enqueued
  {
    const uint4* mask = p.set0.mask;
    if (p.head_to_set != nullptr) {
      const SetDesc sd = p.sets[p.head_to_set[h]];
      mask = sd.mask;
      lists.n = min(sd.row_ptr[1] - sd.row_ptr[0], 2);
      for (int i = 0; i < lists.n; ++i) lists.pr[i] = sd.pairs[sd.row_ptr[0] + i];
    }
    for (int idx = tid; idx < q_rows * 2; idx += blockDim.x) {
      const int row = idx >> 1, tile = idx & 1;
      uint4 bits = make_uint4(0u, 0u, 0u, 0u);
      if (row < p.n_k) {
        for (int i = 0; i < lists.n; ++i)
          if (lists.pr[i].key_tile == tile)
            bits = lists.pr[i].mask_block < 0 ? make_uint4(~0u, ~0u, ~0u, ~0u)
                                              : mask[(size_t)lists.pr[i].mask_block * kBlockM + row];
      }
      uint32_t w[4] = {bits.x, bits.y, bits.z, bits.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {  // cache rows at or past L_k are never live
        const int valid = p.L_k - (tile * kBlockN + i * 32);
        w[i] &= valid >= 32 ? ~0u : (valid <= 0 ? 0u : (1u << valid) - 1u);
      }
      *reinterpret_cast<uint4*>(Ms + row * 8 + tile * 4) = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }

  // ---- everything that does not read Q, K or V happens before the wait, where it overlaps the tail of the
  // previous kernel of the stream: kernel parameters into registers (each first touch of a parameter line is
  // a constant-cache miss), base pointers, zero fill of the padding rows
  const int n_k = p.n_k, L_k = p.L_k;
  const uint16_t* qsrc = p.q + b * p.q_sb + h * p.q_sh + (tid & 7) * 8;
  const uint16_t* ksrc = p.k + b * p.k_sb + h * p.k_sh + (tid & 7) * 8;
  const uint16_t* vsrc = p.v + b * p.v_sb + h * p.v_sh + (tid & 7) * 8;
  uint16_t* obase = p.out + b * p.o_sb + h * p.o_sh;
  int64_t q_st = p.q_st, k_st = p.k_st, v_st = p.v_st, o_st = p.o_st;
  int64_t o_share = (int64_t)p.share_offset * p.o_sb;
  float scale_log2 = p.sm_scale * 1.4426950408889634f;
  asm volatile("" : "+l"(qsrc), "+l"(ksrc), "+l"(vsrc), "+l"(obase));
  asm volatile("" : "+l"(q_st), "+l"(k_st), "+l"(v_st), "+l"(o_st), "+l"(o_share), "+f"(scale_log2));
  {
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
    for (int c = n_k * 8 + tid; c < q_rows * 8; c += blockDim.x)
      *reinterpret_cast<uint4*>(Qs + (c >> 3) * kRowPad + (c & 7) * 8) = zero;
    for (int c = L_k * 8 + tid; c < l_pad * 8; c += blockDim.x) {
      *reinterpret_cast<uint4*>(Ks + (c >> 3) * kRowPad + (c & 7) * 8) = zero;
      *reinterpret_cast<uint4*>(Vs + (c >> 3) * kRowPad + (c & 7) * 8) = zero;
    }
  }

  // ---- stage Q and the K/V prefix (written by earlier work of the stream: wait for it first).  blockDim is a
  // multiple of 32, so a thread keeps its 16-byte column (tid % 8) and walks rows.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if constexpr (KV8) {
    // 8-bit K/V cache (paper Section 4): Q by asynchronous copies as below; the prefix arrives as int8 codes with a
    // scale and a zero point per row and is widened on the way into the same bf16 rows (16 codes per thread and
    // chunk: consecutive threads read consecutive 16 bytes of a row).
    const int row_step = (int)(blockDim.x >> 3);
    uint16_t* qdst = Qs + (tid & 7) * 8;
    for (int row = tid >> 3; row < n_k; row += row_step) cp_async16(qdst + row * kRowPad, qsrc + row * q_st);
    asm volatile("cp.async.commit_group;" ::: "memory");
    const int8_t* kc = p.k8 + b * p.c_sb + h * p.c_sh;
    const int8_t* vc = p.v8 + b * p.c_sb + h * p.c_sh;
    const int64_t zoff = b * p.z_sb + h * p.z_sh;
    for (int c = tid; c < 4 * L_k; c += (int)blockDim.x) {
      const int row = c >> 2, part = c & 3;
      const uint4 kq = __ldg(reinterpret_cast<const uint4*>(kc + (int64_t)row * p.c_st) + part);
      const uint4 vq = __ldg(reinterpret_cast<const uint4*>(vc + (int64_t)row * p.c_st) + part);
      const float ks = __ldg(p.k_scale + zoff + row), kz = __ldg(p.k_zero + zoff + row);
      const float vs = __ldg(p.v_scale + zoff + row), vz = __ldg(p.v_zero + zoff + row);
      uint4 lo, hi;
      widen_codes16(kq, ks, shifted_zero_point(kz, ks), lo, hi);
      *reinterpret_cast<uint4*>(Ks + row * kRowPad + part * 16) = lo;
      *reinterpret_cast<uint4*>(Ks + row * kRowPad + part * 16 + 8) = hi;
      widen_codes16(vq, vs, shifted_zero_point(vz, vs), lo, hi);
      *reinterpret_cast<uint4*>(Vs + row * kRowPad + part * 16) = lo;
      *reinterpret_cast<uint4*>(Vs + row * kRowPad + part * 16 + 8) = hi;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
  } else {
    const int row_step = (int)(blockDim.x >> 3);
    uint16_t* kdst = Ks + (tid & 7) * 8;
    uint16_t* vdst = Vs + (tid & 7) * 8;
    for (int row = tid >> 3; row < L_k; row += row_step) cp_async16(kdst + row * kRowPad, ksrc + row * k_st);
    uint16_t* qdst = Qs + (tid & 7) * 8;
    for (int row = tid >> 3; row < n_k; row += row_step) cp_async16(qdst + row * kRowPad, qsrc + row * q_st);
    asm volatile("cp.async.commit_group;" ::: "memory");
    // V in a group of its own: the scores of the first round are computed while it is still on its way
    for (int row = tid >> 3; row < L_k; row += row_step) cp_async16(vdst + row * kRowPad, vsrc + row * v_st);
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 1;" ::: "memory");
  }
  __syncthreads();

  const int group = warp / SPLIT, part = warp % SPLIT;  // row group; which rounds of it this warp takes
  const int row0 = group * 16;
  if (row0 >= n_k) {  // a warp without query rows only helped staging
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    return;
  }
  bool v_staged = false;

  uint32_t qa[4][4];  // Q fragments of the warp's 16 rows, one per 16 head dimensions
#pragma unroll
  for (int ks = 0; ks < 4; ++ks)
    ldmatrix_x4(qa[ks], Qs + (row0 + (lane & 7) + ((lane >> 3) & 1) * 8) * kRowPad + ks * 16 + (lane >> 4) * 8);

  float o[8][4];
#pragma unroll
  for (int j = 0; j < 8; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
  float lsum[4] = {0.f, 0.f, 0.f, 0.f};  // row sums of P, accumulated by the tensor pipe: P times a block of ones
  float m_run[2] = {-INFINITY, -INFINITY};
  const uint32_t* m_lo = Ms + (row0 + (lane >> 2)) * 8;  // accumulator rows of this lane: lane / 4 and + 8
  const uint32_t* m_hi = m_lo + 64;
  const int n64 = (l_pad + 63) >> 6;
  const int shift = (lane & 3) * 2;  // element (j, e) of a row is key 64 kb + 8 j + 2 (lane % 4) + e
  constexpr uint32_t kOnes = 0x3f803f80u;  // bf16 pair (1, 1)

  for (int kb = part; kb < n64; kb += SPLIT) {  // 64 keys per round
    const uint32_t wl[2] = {m_lo[kb * 2], m_lo[kb * 2 + 1]};
    const uint32_t wh[2] = {m_hi[kb * 2], m_hi[kb * 2 + 1]};
    // 16-key groups with no live key in any of the warp's 16 rows are skipped (also the padding past L_k)
    const uint32_t any[2] = {__reduce_or_sync(0xffffffffu, wl[0] | wh[0]), __reduce_or_sync(0xffffffffu, wl[1] | wh[1])};
    if ((any[0] | any[1]) == 0u) continue;
    bool live[4];
#pragma unroll
    for (int jp = 0; jp < 4; ++jp) live[jp] = ((any[jp >> 1] >> ((jp & 1) * 16)) & 0xffffu) != 0u;
    float s[8][4];
#pragma unroll
    for (int jp = 0; jp < 4; ++jp) {
      s[2 * jp][0] = s[2 * jp][1] = s[2 * jp][2] = s[2 * jp][3] = 0.f;
      s[2 * jp + 1][0] = s[2 * jp + 1][1] = s[2 * jp + 1][2] = s[2 * jp + 1][3] = 0.f;
      if (live[jp]) {
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          uint32_t kf[4];
          ldmatrix_x4(kf, Ks + (kb * 64 + jp * 16 + (lane & 7) + (lane >> 4) * 8) * kRowPad + ks * 16 +
                              ((lane >> 3) & 1) * 8);
          mma_bf16(s[2 * jp], qa[ks], kf[0], kf[1]);
          mma_bf16(s[2 * jp + 1], qa[ks], kf[2], kf[3]);
        }
      }
    }
    // scores of dead keys are removed (groups without a live key are left out altogether)
    const uint32_t bl[2] = {wl[0] >> shift, wl[1] >> shift}, bh[2] = {wh[0] >> shift, wh[1] >> shift};
    float bm[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (live[j >> 1]) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const uint32_t bit = 1u << ((j & 3) * 8 + e);
          s[j][e] = (bl[j >> 2] & bit) ? s[j][e] : -INFINITY;
          s[j][2 + e] = (bh[j >> 2] & bit) ? s[j][2 + e] : -INFINITY;
          bm[0] = fmaxf(bm[0], s[j][e]);
          bm[1] = fmaxf(bm[1], s[j][2 + e]);
        }
      }
    }
    float alpha[2], m_use[2];
#pragma unroll
    for (int x = 0; x < 2; ++x) {  // the four lanes of a quad share a row
      bm[x] = fmaxf(bm[x], __shfl_xor_sync(0xffffffffu, bm[x], 1));
      bm[x] = fmaxf(bm[x], __shfl_xor_sync(0xffffffffu, bm[x], 2));
      const float m_new = fmaxf(m_run[x], bm[x] * scale_log2);
      m_use[x] = m_new == -INFINITY ? 0.f : m_new;  // no live key so far: every p below is 0
      alpha[x] = ex2(m_run[x] - m_use[x]);
      m_run[x] = m_new;
    }
    uint32_t pa[4][4];  // P as A fragments, one per 16 keys
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (live[j >> 1]) {
        pa[j >> 1][(j & 1) * 2] = pack_bf16(ex2(fmaf(s[j][0], scale_log2, -m_use[0])), ex2(fmaf(s[j][1], scale_log2, -m_use[0])));
        pa[j >> 1][(j & 1) * 2 + 1] = pack_bf16(ex2(fmaf(s[j][2], scale_log2, -m_use[1])), ex2(fmaf(s[j][3], scale_log2, -m_use[1])));
      }
    }
    if (!v_staged) {  // second block barrier: once per warp, here or after the loop
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      __syncthreads();
      v_staged = true;
    }
    lsum[0] *= alpha[0];
    lsum[1] *= alpha[0];
    lsum[2] *= alpha[1];
    lsum[3] *= alpha[1];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      o[j][0] *= alpha[0];
      o[j][1] *= alpha[0];
      o[j][2] *= alpha[1];
      o[j][3] *= alpha[1];
    }
#pragma unroll
    for (int jp = 0; jp < 4; ++jp) {
      if (live[jp]) {
        mma_bf16(lsum, pa[jp], kOnes, kOnes);
#pragma unroll
        for (int dn = 0; dn < 4; ++dn) {
          uint32_t vf[4];
          ldmatrix_x4_trans(vf, Vs + (kb * 64 + jp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * kRowPad + dn * 16 +
                                    (lane >> 4) * 8);
          mma_bf16(o[2 * dn], pa[jp], vf[0], vf[1]);
          mma_bf16(o[2 * dn + 1], pa[jp], vf[2], vf[3]);
        }
      }
    }
  }

  if (!v_staged) {  // no live key in any of the warp's rows (the planner rejects such plans): still join the barrier
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
  }

  if (SPLIT == 2) {
    // ---- the pair's second warp hands its partial result (running maximum, row sum, unnormalised output)
    // to the first, which rescales both to the common maximum
    float* Xo = Xs + group * kMergeFloats;
    float* Xm = Xo + 16 * kMergePad;
    float* Xl = Xm + 16;
    const int r_lo = lane >> 2, cq = (lane & 3) * 2;
    if (part == 1) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        *reinterpret_cast<float2*>(Xo + r_lo * kMergePad + j * 8 + cq) = make_float2(o[j][0], o[j][1]);
        *reinterpret_cast<float2*>(Xo + (r_lo + 8) * kMergePad + j * 8 + cq) = make_float2(o[j][2], o[j][3]);
      }
      if ((lane & 3) == 0) {
        Xm[r_lo] = m_run[0];
        Xm[r_lo + 8] = m_run[1];
        Xl[r_lo] = lsum[0];
        Xl[r_lo + 8] = lsum[2];
      }
      __threadfence_block();
      asm volatile("bar.arrive %0, 64;" ::"r"(1 + group) : "memory");
      return;
    }
    asm volatile("bar.sync %0, 64;" ::"r"(1 + group) : "memory");
#pragma unroll
    for (int x = 0; x < 2; ++x) {
      const int row = r_lo + 8 * x;
      const float m1 = Xm[row], l1 = Xl[row];
      const float m_new = fmaxf(m_run[x], m1);
      const float m_use = m_new == -INFINITY ? 0.f : m_new;
      const float a0 = ex2(m_run[x] - m_use), a1 = ex2(m1 - m_use);
      lsum[2 * x] = lsum[2 * x] * a0 + l1 * a1;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float2 o1 = *reinterpret_cast<const float2*>(Xo + row * kMergePad + j * 8 + cq);
        o[j][2 * x] = o[j][2 * x] * a0 + o1.x * a1;
        o[j][2 * x + 1] = o[j][2 * x + 1] * a0 + o1.y * a1;
      }
    }
  }

  // ---- normalise, gather the warp's 16 rows in its (now free) Q rows, store 16 bytes per lane
  const float inv[2] = {1.f / lsum[0], 1.f / lsum[2]};
  __syncwarp();
  {
    uint16_t* r_lo = Qs + (row0 + (lane >> 2)) * kRowPad + (lane & 3) * 2;
    uint16_t* r_hi = r_lo + 8 * kRowPad;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      *reinterpret_cast<uint32_t*>(r_lo + j * 8) = pack_bf16(o[j][0] * inv[0], o[j][1] * inv[0]);
      *reinterpret_cast<uint32_t*>(r_hi + j * 8) = pack_bf16(o[j][2] * inv[1], o[j][3] * inv[1]);
    }
  }
  __syncwarp();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int c = i * 32 + lane;
    const int row = row0 + (c >> 3), part = (c & 7) * 8;
    if (row < n_k) {
      const uint4 v = *reinterpret_cast<const uint4*>(Qs + row * kRowPad + part);
      uint16_t* dst = obase + row * o_st + part;
      *reinterpret_cast<uint4*>(dst) = v;
      if (o_share != 0) *reinterpret_cast<uint4*>(dst + o_share) = v;
    }
  }
}

}  // namespace

bool small_step_candidate(int n_q_tiles, int n_key_tiles, bool raster_only) {
  return raster_only && n_q_tiles == 1 && n_key_tiles >= 1 && n_key_tiles <= 2;
}

int small_step_mode(int n_k, int L_k, long long units, int n_sm) {
  const int warps = (n_k + 15) / 16, rounds = (L_k + 63) / 64;
  // Legacy warp-level mma is several times slower than tcgen05 on this part, so the kernel only wins while
  // the step is a latency chain: up to 18 (16-row warp) x (64-key round) units of work per CTA.  Measured on
  // B200 with 128, 288 and 960 (batch row, head) units: 64 x 155 and 81 x 147 steps are faster here, the
  // 100 x 255 step is faster on the tcgen05 kernel (8.4 against 8.9 us even with two warps per row group).
  if (warps * rounds > 18) return 0;
  // A launch that leaves SMs to spare waits for the chain of rounds of single warps: two warps per row group
  // as soon as there is more than one round (4.8 -> 4.4 us at 36 x 91, 6.9 -> 6.1 us at 64 x 155, 128 units).
  return units <= n_sm && rounds >= 2 ? 2 : 1;
}

template <int SPLIT, bool KV8>
static cudaError_t launch_small_variant(const FwdParams& p, const SmallLists& lists, int n_sm, cudaStream_t stream) {
  static std::once_flag attr_once;
  static cudaError_t attr_err = cudaSuccess;
  constexpr int kMaxSmem = (kBlockM + 2 * 2 * kBlockN) * kRowPad * 2 + kBlockM * 32 +
                           (SPLIT == 2 ? (kBlockM / 16) * kMergeFloats * 4 : 0);
  std::call_once(attr_once, [] {
    attr_err = cudaFuncSetAttribute(fwd_small_kernel<SPLIT, KV8>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
  });
  if (attr_err != cudaSuccess) return attr_err;
  const int q_rows = (p.n_k + 15) / 16 * 16, l_pad = (p.L_k + 15) & ~15;
  // SPLIT warps per 16 query rows; more where the staging copies would otherwise queue up behind few threads,
  // unless the grid fills the SMs several times over (idle warps still hold registers and cost residency)
  int n_warps = q_rows / 16 * SPLIT;
  const int stage_warps = ((q_rows + 2 * l_pad) * 8 + 191) / 192;
  if (n_warps < stage_warps && (long long)p.n_heads * p.batch_computed <= 2LL * n_sm)
    n_warps = stage_warps < kSmallMaxWarps * SPLIT ? stage_warps : kSmallMaxWarps * SPLIT;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)p.n_heads * (unsigned)p.batch_computed);
  cfg.blockDim = dim3((unsigned)n_warps * 32);
  cfg.dynamicSmemBytes = (size_t)(q_rows + 2 * l_pad) * kRowPad * 2 + (size_t)q_rows * 32 +
                         (SPLIT == 2 ? (size_t)(q_rows / 16) * kMergeFloats * 4 : 0);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = p.overlap_launch ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, fwd_small_kernel<SPLIT, KV8>, p, lists);
}

cudaError_t launch_forward_small(const FwdParams& p, const SmallLists& lists, int mode, int n_sm, cudaStream_t stream) {
  return mode == 2 ? launch_small_variant<2, false>(p, lists, n_sm, stream)
                   : launch_small_variant<1, false>(p, lists, n_sm, stream);
}

cudaError_t launch_forward_small_kv8(const FwdParams& p, const SmallLists& lists, int mode, int n_sm,
                                     cudaStream_t stream) {
  return mode == 2 ? launch_small_variant<2, true>(p, lists, n_sm, stream)
                   : launch_small_variant<1, true>(p, lists, n_sm, stream);
}

}  // namespace litevar
