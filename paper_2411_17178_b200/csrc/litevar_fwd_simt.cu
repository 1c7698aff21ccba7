// Plain CUDA-core forward kernel: one warp per query row, fp32 throughout.
//
// It walks the same tile plan and reads the same element-mask blocks as the tensor-core kernel,
// so it cross-checks the plan consumption independently of tcgen05/TMA.  It is slow by design
// (every key row is read from global memory by one lane) and is selected only through
// litevar_plan_set_kernel(LITEVAR_KERNEL_SIMT).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "litevar_internal.h"

namespace litevar {

namespace {

constexpr int kWarpsPerBlock = 4;

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }

// Cache row of slot n of key tile `kt` (any row for a padding slot: its mask bit is never set).
__device__ __forceinline__ int key_slot_row(const FwdParams& p, int kt, int n) {
  if (p.key_geom == nullptr) return kt * kBlockN + n;
  const TileGeom g = p.key_geom[kt];
  if (g.scale < 0) return g.a + n;
  const int s_j = p.patch_scale[g.map_slot];
  return p.patch_off[g.map_slot] + (g.a + n / kPatchCols) * s_j + g.b + n % kPatchCols;
}

__global__ void __launch_bounds__(kWarpsPerBlock * 32) fwd_simt_kernel(FwdParams p) {
  __shared__ float q_sh[kWarpsPerBlock][kHeadDim];
  __shared__ float p_sh[kWarpsPerBlock][kBlockN];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int slot = blockIdx.x * kWarpsPerBlock + warp;  // one warp per query slot of the tile plan
  const int h = blockIdx.y, b = blockIdx.z;
  const int qt = slot / kBlockM, m = slot % kBlockM;
  int q = slot;
  if (p.q_geom != nullptr) {
    const TileGeom g = p.q_geom[qt];
    if (g.scale < 0) {
      q = g.a + m;
    } else {
      const int r = g.a + m / kPatchCols, c = g.b + m % kPatchCols;
      q = (r < p.s_k && c < p.s_k) ? r * p.s_k + c : p.n_k;
    }
  }
  if (q >= p.n_k) return;  // padding slot (whole warp)
  const SetDesc sd = p.head_to_set ? p.sets[p.head_to_set[h]] : p.set0;

  const uint16_t* qrow = p.q + b * p.q_sb + h * p.q_sh + (int64_t)q * p.q_st;
  q_sh[warp][lane] = bf16_bits_to_float(qrow[lane]);
  q_sh[warp][lane + 32] = bf16_bits_to_float(qrow[lane + 32]);
  __syncwarp();

  const uint16_t* kbase = p.k + b * p.k_sb + h * p.k_sh;
  const uint16_t* vbase = p.v + b * p.v_sb + h * p.v_sh;
  float row_max = -INFINITY, row_sum = 0.f, acc0 = 0.f, acc1 = 0.f;

  for (int pi = sd.row_ptr[qt]; pi < sd.row_ptr[qt + 1]; ++pi) {
    const Pair pr = sd.pairs[pi];
    uint4 bits4 = pr.mask_block < 0 ? make_uint4(~0u, ~0u, ~0u, ~0u)
                                    : sd.mask[(size_t)pr.mask_block * kBlockM + m];
    const uint32_t bits[4] = {bits4.x, bits4.y, bits4.z, bits4.w};
    if ((bits[0] | bits[1] | bits[2] | bits[3]) == 0u) continue;
    float s[4];
    float tile_max = -INFINITY;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      s[w] = -INFINITY;
      if ((bits[w] >> lane) & 1u) {
        const uint4* krow =
            reinterpret_cast<const uint4*>(kbase + (int64_t)key_slot_row(p, pr.key_tile, w * 32 + lane) * p.k_st);
        float dot = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          uint4 kk = krow[c];
          const uint32_t u[4] = {kk.x, kk.y, kk.z, kk.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            dot = fmaf(q_sh[warp][c * 8 + 2 * e], __uint_as_float(u[e] << 16), dot);
            dot = fmaf(q_sh[warp][c * 8 + 2 * e + 1], __uint_as_float(u[e] & 0xffff0000u), dot);
          }
        }
        s[w] = dot * p.sm_scale;
        tile_max = fmaxf(tile_max, s[w]);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) tile_max = fmaxf(tile_max, __shfl_xor_sync(0xffffffffu, tile_max, o));
    const float new_max = fmaxf(row_max, tile_max);  // finite: the tile has at least one live key
    const float alpha = row_max == -INFINITY ? 0.f : __expf(row_max - new_max);
    float psum = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      float pv = s[w] == -INFINITY ? 0.f : __expf(s[w] - new_max);
      p_sh[warp][w * 32 + lane] = pv;
      psum += pv;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, o);
    row_sum = row_sum * alpha + psum;
    acc0 *= alpha;
    acc1 *= alpha;
    row_max = new_max;
    __syncwarp();
    for (int w = 0; w < 4; ++w) {
      uint32_t bw = bits[w];
      while (bw) {
        int n = __ffs(bw) - 1;
        bw &= bw - 1;
        float pv = p_sh[warp][w * 32 + n];
        uint32_t vv = *reinterpret_cast<const uint32_t*>(
            vbase + (int64_t)key_slot_row(p, pr.key_tile, w * 32 + n) * p.v_st + 2 * lane);
        acc0 = fmaf(pv, __uint_as_float(vv << 16), acc0);
        acc1 = fmaf(pv, __uint_as_float(vv & 0xffff0000u), acc1);
      }
    }
    __syncwarp();
  }
  const float inv = 1.f / row_sum;
  __nv_bfloat162 o2 = __floats2bfloat162_rn(acc0 * inv, acc1 * inv);
  uint16_t* orow = p.out + b * p.o_sb + h * p.o_sh + (int64_t)q * p.o_st;
  *reinterpret_cast<__nv_bfloat162*>(orow + 2 * lane) = o2;
  if (p.share_offset > 0) {
    uint16_t* orow2 = p.out + (int64_t)(b + p.share_offset) * p.o_sb + h * p.o_sh + (int64_t)q * p.o_st;
    *reinterpret_cast<__nv_bfloat162*>(orow2 + 2 * lane) = o2;
  }
}

}  // namespace

cudaError_t launch_forward_simt(const FwdParams& p, int n_q_tiles, cudaStream_t stream) {
  dim3 grid((unsigned)(n_q_tiles * (kBlockM / kWarpsPerBlock)), (unsigned)p.n_heads,
            (unsigned)p.batch_computed);
  fwd_simt_kernel<<<grid, kWarpsPerBlock * 32, 0, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace litevar
