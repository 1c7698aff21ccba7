// litevar_attn_forward_static: step-k attention for callers that cannot allocate device memory.
//
// The plan API (litevar_attn_plan) calls cudaMalloc for its tile lists and mask blocks.  Some callers
// cannot: code that runs inside a fixed memory budget handed out at start-up, a plug-in that must not
// touch the allocator of its host process, or a call site that is reached while allocation is forbidden
// (for example between other libraries' captured work).  For them this entry point builds the tile plan
// of ONE step on the device into a file-scope array that ships with the library and then runs the same
// tensor-core forward kernel on it.  It calls no cudaMalloc, no cudaFree and no allocating library
// routine.  Price: the array has a fixed size (steps with more than kStaticMaxPairs candidate tile pairs
// are refused), every GPU that loads the library holds it until the process exits, every call shares it,
// and the plan is rebuilt on every call (two small extra launches).
#include <cuda_runtime.h>

#include <mutex>

#include "litevar_internal.h"

namespace litevar {

namespace {

constexpr int kStaticMaxPairs = 2048;  // candidate (query tile, key tile) pairs of one step
constexpr int kStaticMaxDevices = 64;

// Everything one step's plan needs, at fixed offsets.  Mask block c belongs to candidate pair c
// (query tile c / n_key_tiles, key tile c % n_key_tiles), so no second compaction is needed.
struct StaticPlan {
  SetDesc set;      // read by the forward kernel through FwdParams::sets
  int32_t status;   // bounded-wait flag of the forward kernel; cleared at the start of every call
  int32_t pad[9];
  int32_t row_ptr[kStaticMaxPairs + 1];
  Pair pairs[kStaticMaxPairs];
  uint8_t cls[kStaticMaxPairs];
  uint4 mask[(size_t)kStaticMaxPairs * kBlockM];
};

// 4.2 MB per GPU.  In host code this name is only a handle for cudaGetSymbolAddress: it is not a device
// address and must never be passed to a kernel.  Device code below names it directly.
static __device__ __align__(256) unsigned char litevar_static_scratch[sizeof(StaticPlan)];

struct StepArgs {
  int32_t k0, s_k, n_k, L_k, n_q_tiles, n_key_tiles, shape;
  int32_t radius[kMaxScales];  // radius of key scale j at this step, -1 = whole part live
};

__device__ __forceinline__ StaticPlan* static_plan() { return reinterpret_cast<StaticPlan*>(litevar_static_scratch); }

// One block per candidate pair: thread m owns query slot m, evaluates the window predicate of
// paper Section 2 against the 128 key slots of the key tile, writes its 128 mask bits and the
// class of the pair (0 dead, 1 partial, 2 full).
__global__ void __launch_bounds__(kBlockM) static_classify_kernel(Schedule sc, StepArgs a) {
  __shared__ int16_t ks_j[kBlockN], ks_r[kBlockN], ks_c[kBlockN];
  __shared__ int32_t ks_t[kBlockN];
  StaticPlan* sp = static_plan();
  const int kt = blockIdx.x, qt = blockIdx.y, m = threadIdx.x;
  {
    const int t = kt * kBlockN + m;
    int j = -1, r = 0, c = 0, tin = 0;
    if (t < a.L_k) {
      j = 0;
      while (t >= sc.off[j + 1]) ++j;
      tin = t - sc.off[j];
      r = tin / sc.scale[j];
      c = tin - r * sc.scale[j];
    }
    ks_j[m] = (int16_t)j;
    ks_r[m] = (int16_t)r;
    ks_c[m] = (int16_t)c;
    ks_t[m] = tin;
  }
  __syncthreads();
  const int q = qt * kBlockM + m;
  const bool valid = q < a.n_k;
  uint32_t w[4] = {0u, 0u, 0u, 0u};
  if (valid) {
    const int r = q / a.s_k, c = q - r * a.s_k;
    int cur = -2, rad = -1, rlo = 0, rhi = -1, clo = 0, chi = -1;
    long long band_ctr = 0;
    for (int n = 0; n < kBlockN; ++n) {
      const int j = ks_j[n];
      if (j < 0) break;  // slots past L_k are the tail of the last tile
      if (j != cur) {
        cur = j;
        rad = a.radius[j];
        const int s_j = sc.scale[j];
        if (a.shape == LITEVAR_WINDOW_SQUARE) {
          const int cr = ((2 * r + 1) * s_j) / (2 * a.s_k), cc = ((2 * c + 1) * s_j) / (2 * a.s_k);
          rlo = max(0, cr - rad); rhi = min(s_j - 1, cr + rad);
          clo = max(0, cc - rad); chi = min(s_j - 1, cc + rad);
        } else {
          band_ctr = ((2LL * q + 1) * s_j * s_j) / (2LL * a.n_k);
        }
      }
      bool lv;
      if (rad < 0) {
        lv = true;
      } else if (a.shape == LITEVAR_WINDOW_SQUARE) {
        lv = ks_r[n] >= rlo && ks_r[n] <= rhi && ks_c[n] >= clo && ks_c[n] <= chi;
      } else {
        const long long d = (long long)ks_t[n] - band_ctr;
        lv = d <= rad && -d <= rad;
      }
      if (lv) w[n >> 5] |= 1u << (n & 31);
    }
  }
  const int cnt = __popc(w[0]) + __popc(w[1]) + __popc(w[2]) + __popc(w[3]);
  const int any = __syncthreads_or(cnt != 0);
  const int all = __syncthreads_and(!valid || cnt == kBlockN);
  const int cand = qt * a.n_key_tiles + kt;
  sp->mask[(size_t)cand * kBlockM + m] = make_uint4(w[0], w[1], w[2], w[3]);
  if (m == 0) sp->cls[cand] = any ? (all ? 2 : 1) : 0;
}

// One block: per query tile count the live pairs, scan, write the CSR list in canonical order
// (query tile ascending, key tile ascending), publish the descriptor and clear the status word.
__global__ void static_compact_kernel(int n_q_tiles, int n_key_tiles) {
  __shared__ int32_t count[kStaticMaxPairs];
  StaticPlan* sp = static_plan();
  for (int qt = threadIdx.x; qt < n_q_tiles; qt += blockDim.x) {
    int l = 0;
    for (int kt = 0; kt < n_key_tiles; ++kt) l += sp->cls[qt * n_key_tiles + kt] != 0;
    count[qt] = l;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int acc = 0;
    for (int qt = 0; qt < n_q_tiles; ++qt) {
      sp->row_ptr[qt] = acc;
      acc += count[qt];
    }
    sp->row_ptr[n_q_tiles] = acc;
    sp->set.row_ptr = sp->row_ptr;
    sp->set.pairs = sp->pairs;
    sp->set.mask = sp->mask;
    sp->status = 0;
  }
  __syncthreads();
  for (int qt = threadIdx.x; qt < n_q_tiles; qt += blockDim.x) {
    int o = sp->row_ptr[qt];
    for (int kt = 0; kt < n_key_tiles; ++kt) {
      const int cand = qt * n_key_tiles + kt;
      const int c = sp->cls[cand];
      if (c != 0) {
        sp->pairs[o].key_tile = kt;
        sp->pairs[o].mask_block = c == 1 ? cand : -1;
        ++o;
      }
    }
  }
}

// Device address of the array on the current device, looked up once per device.
litevar_status_t static_plan_address(StaticPlan** out) {
  static std::mutex mu;
  static StaticPlan* addr[kStaticMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    (void)cudaGetLastError();
    return LITEVAR_ERR_CUDA;
  }
  if (dev < 0 || dev >= kStaticMaxDevices) return LITEVAR_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(mu);
  if (!addr[dev]) {
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
      (void)cudaGetLastError();
      return LITEVAR_ERR_CUDA;
    }
    if (prop.major != 10) return LITEVAR_ERR_ARCH;
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, litevar_static_scratch) != cudaSuccess || !ptr) {
      (void)cudaGetLastError();
      return LITEVAR_ERR_CUDA;
    }
    addr[dev] = static_cast<StaticPlan*>(ptr);
  }
  *out = addr[dev];
  return LITEVAR_OK;
}

bool strides_valid(const litevar_strides_t* s) {
  return s && s->batch >= 0 && s->head >= 0 && s->token >= kHeadDim && (s->batch % 8) == 0 && (s->head % 8) == 0 &&
         (s->token % 8) == 0;
}

}  // namespace

}  // namespace litevar

using namespace litevar;

extern "C" litevar_status_t litevar_attn_forward_static(
    const int32_t* scales, int32_t n_scales, int32_t n_heads, int32_t head_dim, float sm_scale,
    const litevar_window_t* window, int32_t share_cfg, int32_t step_k, int32_t batch_pairs, const void* Q,
    const litevar_strides_t* sq, const void* Kc, const litevar_strides_t* sk, const void* Vc,
    const litevar_strides_t* sv, void* out, const litevar_strides_t* so, void* stream_) {
  if (!scales || !window || !Q || !Kc || !Vc || !out) return LITEVAR_ERR_INVALID_ARG;
  if (n_scales < 1 || n_scales > kMaxScales || n_heads < 1 || head_dim < 1) return LITEVAR_ERR_INVALID_ARG;
  for (int i = 0; i < n_scales; ++i)
    if (scales[i] < 1 || scales[i] > kMaxScale) return LITEVAR_ERR_INVALID_ARG;
  if (step_k < 1 || step_k > n_scales || batch_pairs < 1) return LITEVAR_ERR_INVALID_ARG;
  if (window->shape != LITEVAR_WINDOW_SQUARE && window->shape != LITEVAR_WINDOW_BAND) return LITEVAR_ERR_INVALID_ARG;
  if (!window->radius && (window->rho_den <= 0 || window->rho_num < 0 || window->n_global_scales < 0))
    return LITEVAR_ERR_INVALID_ARG;
  if (!strides_valid(sq) || !strides_valid(sk) || !strides_valid(sv) || !strides_valid(so))
    return LITEVAR_ERR_INVALID_ARG;
  if (((uintptr_t)Q | (uintptr_t)Kc | (uintptr_t)Vc | (uintptr_t)out) & 15) return LITEVAR_ERR_INVALID_ARG;
  if (head_dim != kHeadDim || window->n_sets != 1) return LITEVAR_ERR_UNSUPPORTED;

  Schedule sc = {};
  sc.n_scales = n_scales;
  for (int i = 0; i < n_scales; ++i) {
    sc.scale[i] = scales[i];
    sc.off[i + 1] = sc.off[i] + scales[i] * scales[i];
  }
  StepArgs a = {};
  a.k0 = step_k - 1;
  a.s_k = scales[a.k0];
  a.n_k = a.s_k * a.s_k;
  a.L_k = sc.off[step_k];
  a.n_q_tiles = (a.n_k + kBlockM - 1) / kBlockM;
  a.n_key_tiles = (a.L_k + kBlockN - 1) / kBlockN;
  a.shape = window->shape;
  // the step must fit the fixed array
  if ((long long)a.n_q_tiles * a.n_key_tiles > kStaticMaxPairs) return LITEVAR_ERR_UNSUPPORTED;
  for (int j = 0; j < kMaxScales; ++j) a.radius[j] = -1;
  for (int j = 0; j <= a.k0; ++j) {
    int w;
    if (window->radius) {
      w = window->radius[(size_t)a.k0 * n_scales + j];
      if (w < 0) w = -1;
    } else if (j < window->n_global_scales) {
      w = -1;
    } else {
      const long long ext = a.shape == LITEVAR_WINDOW_BAND ? (long long)scales[j] * scales[j] : scales[j];
      w = (int)((2LL * window->rho_num * ext + window->rho_den) / (2LL * window->rho_den));
    }
    a.radius[j] = w;
  }

  StaticPlan* sp = nullptr;
  litevar_status_t st = static_plan_address(&sp);
  if (st != LITEVAR_OK) return st;

  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  dim3 grid((unsigned)a.n_key_tiles, (unsigned)a.n_q_tiles);
  static_classify_kernel<<<grid, kBlockM, 0, stream>>>(sc, a);
  static_compact_kernel<<<1, 256, 0, stream>>>(a.n_q_tiles, a.n_key_tiles);
  if (cudaGetLastError() != cudaSuccess) return LITEVAR_ERR_CUDA;

  FwdParams p;
  p.sets = &sp->set;
  p.head_to_set = nullptr;
  p.set0 = SetDesc{sp->row_ptr, sp->pairs, sp->mask};  // device addresses inside the fixed array
  p.order = nullptr;
  p.q = static_cast<const uint16_t*>(Q);
  p.k = static_cast<const uint16_t*>(Kc);
  p.v = static_cast<const uint16_t*>(Vc);
  p.out = static_cast<uint16_t*>(out);
  p.q_sb = sq->batch; p.q_sh = sq->head; p.q_st = sq->token;
  p.k_sb = sk->batch; p.k_sh = sk->head; p.k_st = sk->token;
  p.v_sb = sv->batch; p.v_sh = sv->head; p.v_st = sv->token;
  p.o_sb = so->batch; p.o_sh = so->head; p.o_st = so->token;
  p.n_k = a.n_k;
  p.L_k = a.L_k;
  p.n_heads = n_heads;
  p.q_geom = nullptr;  // raster tiles
  p.key_geom = nullptr;
  p.s_k = a.s_k;
  p.q_patch = 0;
  p.raster_len = a.L_k;
  p.first_patch = step_k;
  p.n_patch_scales = 0;
  for (int i = 0; i < kMaxPatchScales; ++i) p.patch_scale[i] = p.patch_off[i] = 0;
  p.batch_computed = share_cfg ? batch_pairs : 2 * batch_pairs;
  p.share_offset = share_cfg ? batch_pairs : 0;
  p.sm_scale = sm_scale > 0.f ? sm_scale : 0.125f;
  p.status = &sp->status;
  p.pairs_per_tile = 0;
  p.units_per_group = units_per_l2_group(p.L_k, p.n_heads * p.batch_computed);
  p.first_tile_zero = 0;
  p.overlap_launch = 0;  // the plan is written by the two kernels launched just above
  return launch_forward_tcgen05(p, a.n_q_tiles, stream);
}
