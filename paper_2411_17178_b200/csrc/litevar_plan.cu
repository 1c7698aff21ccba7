// Host side of the C ABI and the device-side mask planner.
//
// The planner turns the window definition of the paper's Section 2 (one window per part of the
// step-k attention map, the first parts global) into, per step, a CSR list of live
// (query tile, key tile) pairs plus a 128x128-bit element mask for every partially live pair.
// Everything that depends on the mask geometry happens here; the attention kernels only walk
// the list and apply the bit masks, so they are independent of the window shape.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <new>

#include "litevar_internal.h"

using namespace litevar;

namespace {

#define LV_CUDA(expr)                          \
  do {                                         \
    cudaError_t e__ = (expr);                  \
    if (e__ != cudaSuccess) {                  \
      (void)cudaGetLastError();                \
      return e__ == cudaErrorMemoryAllocation ? LITEVAR_ERR_OOM : LITEVAR_ERR_CUDA; \
    }                                          \
  } while (0)

// ------------------------------------------------------------------ A1: window table
// radius[k][j] for step k+1 and key scale j+1 (0-based indices here); -1 = whole part live.
// Default rule: scales j <= n_global are global; otherwise round-half-up of rho * s_j (SQUARE)
// or rho * n_j (BAND).  A caller table is copied, with unused entries (j > k) set to -1.
__global__ void window_table_kernel(Schedule sc, int shape, int n_global, int rho_num, int rho_den,
                                    const int32_t* user, int32_t* radius) {
  int K = sc.n_scales;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < K * K; i += gridDim.x * blockDim.x) {
    int k = i / K, j = i % K;
    int w;
    if (j > k) {
      w = -1;
    } else if (user != nullptr) {
      w = user[i] < 0 ? -1 : user[i];
    } else if (j < n_global) {
      w = -1;
    } else {
      long long ext = shape == LITEVAR_WINDOW_BAND ? (long long)sc.scale[j] * sc.scale[j] : sc.scale[j];
      w = (int)((2LL * rho_num * ext + rho_den) / (2LL * rho_den));
    }
    radius[i] = w;
  }
}

// ------------------------------------------------------------------ A2: per-axis bounds
// For query row (or column) x of scale k and key scale j: the key cell containing the centre of
// cell x is ctr = floor((2x+1) s_j / (2 s_k)); the live interval is [ctr-w, ctr+w] clipped to the grid.
__global__ void bounds_kernel(Schedule sc, int k0, const int32_t* radius_row, int2* bounds) {
  int s_k = sc.scale[k0];
  int total = (k0 + 1) * s_k;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    int j = i / s_k, x = i % s_k;
    int s_j = sc.scale[j];
    int w = radius_row[j];
    int2 b;
    if (w < 0) {
      b = make_int2(0, s_j - 1);
    } else {
      int ctr = ((2 * x + 1) * s_j) / (2 * s_k);
      b = make_int2(max(0, ctr - w), min(s_j - 1, ctr + w));
    }
    bounds[i] = b;
  }
}

// ------------------------------------------------------------------ element predicate over one tile pair
struct PlanGeom {
  int k0;           // 0-based step
  int s_k, n_k, L_k;
  int n_key_tiles;
  int shape;
  int raster_len;             // cache rows covered by raster key tiles
  const TileGeom* q_geom;     // [n_q_tiles]
  const TileGeom* key_geom;   // [n_key_tiles]
};

// Query token (within the current scale) of slot m of a query tile, or -1 for a padding slot.
__device__ __forceinline__ int query_slot_token(const TileGeom& g, int m, int s_k, int n_k, int& r, int& c) {
  if (g.scale < 0) {
    int q = g.a + m;
    if (q >= n_k) return -1;
    r = q / s_k;
    c = q - r * s_k;
    return q;
  }
  r = g.a + m / kPatchCols;
  c = g.b + m % kPatchCols;
  if (r >= s_k || c >= s_k) return -1;
  return r * s_k + c;
}

// Live bits of query slot `m` of query tile `qt` against the 128 key slots of key tile `kt`.
// Must be called by all 128 threads of the block (fills shared key-slot tables).  `q_out` receives the
// query token of the slot (-1: padding slot, all bits zero).
__device__ uint4 tile_row_bits(const Schedule& sc, const PlanGeom& g, const int2* __restrict__ bounds,
                               const int32_t* __restrict__ radius_row, int qt, int kt,
                               int16_t* ks_j, int16_t* ks_r, int16_t* ks_c, int32_t* ks_t, int& q_out) {
  int m = threadIdx.x;
  {
    const TileGeom kg = g.key_geom[kt];
    int j = -1, r = 0, c = 0, tin = 0;
    if (kg.scale < 0) {
      int t = kg.a + m;  // raster key tile: slot n is cache row a + n, inside the raster prefix
      if (t < g.raster_len) {
        j = 0;
        while (t >= sc.off[j + 1]) ++j;
        tin = t - sc.off[j];
        r = tin / sc.scale[j];
        c = tin % sc.scale[j];
      }
    } else {
      int s_j = sc.scale[kg.scale];
      r = kg.a + m / kPatchCols;
      c = kg.b + m % kPatchCols;
      if (r < s_j && c < s_j) {
        j = kg.scale;
        tin = r * s_j + c;
      }
    }
    ks_j[m] = (int16_t)j;
    ks_r[m] = (int16_t)r;
    ks_c[m] = (int16_t)c;
    ks_t[m] = tin;
  }
  __syncthreads();
  int r = 0, c = 0;
  const int q = query_slot_token(g.q_geom[qt], m, g.s_k, g.n_k, r, c);
  q_out = q;
  uint32_t w[4] = {0u, 0u, 0u, 0u};
  if (q >= 0) {
    int cur_j = -2;
    int2 br = make_int2(0, -1), bc = make_int2(0, -1);
    long long band_ctr = 0;
    int band_w = -1;
    for (int n = 0; n < kBlockN; ++n) {
      int j = ks_j[n];
      bool lv = false;
      if (j >= 0) {
        if (j != cur_j) {
          cur_j = j;
          if (g.shape == LITEVAR_WINDOW_SQUARE) {
            br = bounds[j * g.s_k + r];
            bc = bounds[j * g.s_k + c];
          } else {
            band_w = radius_row[j];
            long long n_j = (long long)sc.scale[j] * sc.scale[j];
            band_ctr = ((2LL * q + 1) * n_j) / (2LL * g.n_k);
          }
        }
        if (g.shape == LITEVAR_WINDOW_SQUARE) {
          int kr = ks_r[n], kc = ks_c[n];
          lv = kr >= br.x && kr <= br.y && kc >= bc.x && kc <= bc.y;
        } else {
          long long d = (long long)ks_t[n] - band_ctr;
          lv = band_w < 0 || (d <= band_w && -d <= band_w);
        }
      }
      if (lv) w[n >> 5] |= 1u << (n & 31);
    }
  }
  __syncthreads();
  return make_uint4(w[0], w[1], w[2], w[3]);
}

// ------------------------------------------------------------------ A3 pass 1: classify every candidate pair
// cls: 0 dead, 1 partial, 2 full (every valid query slot sees all 128 key slots live).
__global__ void __launch_bounds__(128) classify_kernel(Schedule sc, PlanGeom g, const int2* bounds,
                                                       const int32_t* radius_row, uint8_t* cls,
                                                       int32_t* row_live, unsigned long long* live_entries) {
  __shared__ int16_t ks_j[kBlockN], ks_r[kBlockN], ks_c[kBlockN];
  __shared__ int32_t ks_t[kBlockN];
  int kt = blockIdx.x, qt = blockIdx.y;
  int q;
  uint4 b = tile_row_bits(sc, g, bounds, radius_row, qt, kt, ks_j, ks_r, ks_c, ks_t, q);
  bool valid = q >= 0;
  int cnt = __popc(b.x) + __popc(b.y) + __popc(b.z) + __popc(b.w);
  int any = __syncthreads_or(cnt != 0);
  int all = __syncthreads_and(!valid || cnt == kBlockN);
  if (valid && cnt) atomicAdd(&row_live[q], cnt);
  // block total
  for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
  if ((threadIdx.x & 31) == 0 && cnt) atomicAdd(live_entries, (unsigned long long)cnt);
  if (threadIdx.x == 0) cls[qt * g.n_key_tiles + kt] = any ? (all ? 2 : 1) : 0;
}

// ------------------------------------------------------------------ A3 pass 2: count + exclusive scan
// One block; thread qt counts the live and partial pairs of query tile qt, then a serial scan
// (at most 512 tiles) writes the CSR offsets.  totals = {pairs, partial, full}.
__global__ void count_scan_kernel(int n_q_tiles, int n_key_tiles, const uint8_t* cls, int32_t* row_ptr,
                                  int32_t* partial_base, int32_t* totals) {
  extern __shared__ int32_t sh[];
  int32_t* nl = sh;
  int32_t* np = sh + n_q_tiles;
  for (int qt = threadIdx.x; qt < n_q_tiles; qt += blockDim.x) {
    int l = 0, p = 0;
    for (int kt = 0; kt < n_key_tiles; ++kt) {
      int c = cls[qt * n_key_tiles + kt];
      l += c != 0;
      p += c == 1;
    }
    nl[qt] = l;
    np[qt] = p;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int al = 0, ap = 0;
    for (int qt = 0; qt < n_q_tiles; ++qt) {
      row_ptr[qt] = al;
      partial_base[qt] = ap;
      al += nl[qt];
      ap += np[qt];
    }
    row_ptr[n_q_tiles] = al;
    totals[0] = al;
    totals[1] = ap;
    totals[2] = al - ap;
  }
}

// ------------------------------------------------------------------ A3 pass 3: compact in canonical order
__global__ void compact_kernel(int n_q_tiles, int n_key_tiles, const uint8_t* cls, const int32_t* row_ptr,
                               const int32_t* partial_base, Pair* pairs, int32_t* mask_block_of) {
  int qt = blockIdx.x * blockDim.x + threadIdx.x;
  if (qt >= n_q_tiles) return;
  int o = row_ptr[qt], pb = partial_base[qt];
  for (int kt = 0; kt < n_key_tiles; ++kt) {
    int c = cls[qt * n_key_tiles + kt];
    int blk = -1;
    if (c == 1) blk = pb++;
    mask_block_of[qt * n_key_tiles + kt] = blk;
    if (c != 0) {
      pairs[o].key_tile = kt;
      pairs[o].mask_block = blk;
      ++o;
    }
  }
}

// ------------------------------------------------------------------ A3 pass 4: element masks of partial pairs
__global__ void __launch_bounds__(128) mask_bits_kernel(Schedule sc, PlanGeom g, const int2* bounds,
                                                        const int32_t* radius_row, const int32_t* mask_block_of,
                                                        uint4* mask) {
  __shared__ int16_t ks_j[kBlockN], ks_r[kBlockN], ks_c[kBlockN];
  __shared__ int32_t ks_t[kBlockN];
  int kt = blockIdx.x, qt = blockIdx.y;
  int blk = mask_block_of[qt * g.n_key_tiles + kt];
  if (blk < 0) return;  // uniform per block
  int q;
  uint4 b = tile_row_bits(sc, g, bounds, radius_row, qt, kt, ks_j, ks_r, ks_c, ks_t, q);
  mask[(size_t)blk * kBlockM + threadIdx.x] = b;
}

// Launch order of the CTAs of the forward kernel (one CTA = query tiles 2u and 2u+1): heaviest first, so
// that the light corner tiles fill the tail of the grid.  Rank sort, one thread per CTA.
__global__ void launch_order_kernel(int n_q_tiles, const int32_t* row_ptr, int32_t* order) {
  const int n = (n_q_tiles + 1) / 2;
  const int u = blockIdx.x * blockDim.x + threadIdx.x;
  if (u >= n) return;
  auto work = [&](int v) { return row_ptr[min(2 * v + 2, n_q_tiles)] - row_ptr[2 * v]; };
  const int mine = work(u);
  int rank = 0;
  for (int v = 0; v < n; ++v) {
    const int wv = work(v);
    rank += (wv > mine) || (wv == mine && v < u);
  }
  order[rank] = u;
}

// Does every query tile list key tile 0 first?  (It does whenever the first cache rows stay live for every
// query, as under any window of the paper: the coarsest scales are global.)  The forward kernel then starts
// the copies of that tile before it has read anything of the plan.
__global__ void first_tile_kernel(int n_q_tiles, const int32_t* row_ptr, const Pair* pairs, int32_t* not_zero) {
  const int qt = blockIdx.x * blockDim.x + threadIdx.x;
  if (qt >= n_q_tiles) return;
  const int b = row_ptr[qt], e = row_ptr[qt + 1];
  if (e == b || pairs[b].key_tile != 0) atomicExch(not_zero, 1);
}

__global__ void empty_row_kernel(int n_k, const int32_t* row_live, int32_t* flag) {
  int q = blockIdx.x * blockDim.x + threadIdx.x;
  if (q < n_k && row_live[q] == 0) atomicExch(flag, 1);
}

// ------------------------------------------------------------------ debug: dense mask from the tile plan
__global__ void __launch_bounds__(128) materialize_kernel(SetDesc sd, Schedule sc, PlanGeom g, uint32_t* dense) {
  int qt = blockIdx.x, m = threadIdx.x;
  int r, c;
  const int q = query_slot_token(g.q_geom[qt], m, g.s_k, g.n_k, r, c);
  if (q < 0) return;
  int words = (g.L_k + 31) / 32;
  for (int p = sd.row_ptr[qt]; p < sd.row_ptr[qt + 1]; ++p) {
    Pair pr = sd.pairs[p];
    uint4 b = pr.mask_block < 0 ? make_uint4(~0u, ~0u, ~0u, ~0u)
                                : sd.mask[(size_t)pr.mask_block * kBlockM + m];
    uint32_t w[4] = {b.x, b.y, b.z, b.w};
    const TileGeom kg = g.key_geom[pr.key_tile];
    for (int n = 0; n < kBlockN; ++n) {
      if (!((w[n >> 5] >> (n & 31)) & 1u)) continue;
      int t;
      if (kg.scale < 0) {
        t = kg.a + n;
        if (t >= g.raster_len) continue;
      } else {
        int s_j = sc.scale[kg.scale];
        int kr = kg.a + n / kPatchCols, kc = kg.b + n % kPatchCols;
        if (kr >= s_j || kc >= s_j) continue;
        t = sc.off[kg.scale] + kr * s_j + kc;
      }
      dense[(size_t)q * words + (t >> 5)] |= 1u << (t & 31);  // row q belongs to this thread alone
    }
  }
}

// Bump allocator over one device allocation: sizes are added up in a first pass (base == nullptr), the block is
// allocated, and the same sequence of calls then hands out the pointers.  256-byte granules.
struct Arena {
  char* base = nullptr;
  size_t used = 0;
  template <typename T>
  T* take(size_t count) {
    const size_t bytes = (count * sizeof(T) + 255) & ~static_cast<size_t>(255);
    T* p = base ? reinterpret_cast<T*>(base + used) : nullptr;
    used += bytes ? bytes : 256;
    return p;
  }
};

// Scratch of one (step, window set) during planning.
struct SetScratch {
  uint8_t* cls = nullptr;
  int32_t *row_live = nullptr, *partial_base = nullptr, *blk = nullptr;
};

// Per (step, set) results the host needs: written by the planner kernels into one device array, read back once.
struct SetTotals {
  int32_t n_pairs, n_partial, n_full, empty_row;  // count_scan_kernel / empty_row_kernel
  unsigned long long live_entries;                // classify_kernel
  int32_t first_not_zero, pad;                    // first_tile_kernel
  Pair first_pairs[2];                            // the whole list of a small step (n_pairs <= 2)
};

__global__ void copy_first_pairs_kernel(const Pair* pairs, const int32_t* n_pairs, Pair* out) {
  if (threadIdx.x < 2 && (int)threadIdx.x < *n_pairs) out[threadIdx.x] = pairs[threadIdx.x];
}

// The plan's buffers, the tensor maps and the launch all belong to the device the plan was made on.
bool on_plan_device(const litevar_plan_t* plan) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    (void)cudaGetLastError();
    return false;
  }
  return dev == plan->device;
}

bool strides_ok(const litevar_strides_t* s) {
  return s && s->batch >= 0 && s->head >= 0 && s->token >= kHeadDim && (s->batch % 8) == 0 &&
         (s->head % 8) == 0 && (s->token % 8) == 0;
}

// How the small-step kernel would run this step for `units` (batch row, head) units: 0 = not at all.
int small_mode(const litevar_plan_t* plan, const Step& st, long long units) {
  if (plan->kernel != LITEVAR_KERNEL_AUTO) return 0;
  for (const StepSet& ss : st.sets)  // every window set of the step has a list the small-step kernel can take
    if (ss.small.n <= 0) return 0;
  return small_step_mode(st.n_k, st.L_k, units, plan->n_sm);
}

#define LV_TRY(expr)                                                                              \
  do {                                                                                            \
    cudaError_t e__ = (expr);                                                                     \
    if (e__ != cudaSuccess) {                                                                     \
      (void)cudaGetLastError();                                                                   \
      return e__ == cudaErrorMemoryAllocation ? LITEVAR_ERR_OOM : LITEVAR_ERR_CUDA;               \
    }                                                                                             \
  } while (0)

// Everything litevar_attn_plan does after its argument checks.  Device memory: one arena for the plan (tables,
// tile geometry, bounds, lists, launch orders; the lists sized for every candidate pair), one block for the
// element masks (sized exactly, once the device has counted the partial pairs) and one scratch block that is
// freed before returning.  Two synchronisations: after the counting pass (the mask block's size and the
// empty-row check come from it) and at the end.
litevar_status_t build_plan(litevar_plan* plan, const int32_t* scales, int32_t n_scales, int32_t n_heads, float sm_scale,
                            const litevar_window_t* window, const litevar_cfg_share_t* share, int dev, int n_sm,
                            cudaStream_t stream) {
  plan->device = dev;
  plan->n_sm = n_sm;
  plan->n_heads = n_heads;
  plan->n_sets = window->n_sets;
  plan->shape = window->shape;
  plan->n_global = window->n_global_scales;
  plan->rho_num = window->rho_num;
  plan->rho_den = window->rho_den;
  plan->tiling = window->tiling;
  plan->sm_scale = sm_scale > 0.f ? sm_scale : 0.125f;
  Schedule& sc = plan->sched;
  memset(&sc, 0, sizeof(sc));
  sc.n_scales = n_scales;
  for (int i = 0; i < n_scales; ++i) {
    sc.scale[i] = scales[i];
    sc.off[i + 1] = sc.off[i] + scales[i] * scales[i];
  }
  const int K = n_scales, n_sets = plan->n_sets;
  if (window->head_to_set && n_sets > 1) plan->head_to_set.assign(window->head_to_set, window->head_to_set + n_heads);

  // ---- tile geometry of every step (host): raster tiles of 128 consecutive tokens, or 8x16 patches of a scale's
  // grid where the grid is large enough for a 2-D window to leave whole patches dead
  plan->steps.resize(K);
  for (int k0 = 0; k0 < K; ++k0) {
    Step& st = plan->steps[k0];
    st.s_k = sc.scale[k0];
    st.n_k = st.s_k * st.s_k;
    st.L_k = sc.off[k0 + 1];
    // AUTO: patches pay off for 2-D (square) windows on large grids; a band in token order wants raster tiles
    const bool auto_patch = plan->tiling == LITEVAR_TILING_AUTO && plan->shape == LITEVAR_WINDOW_SQUARE;
    const int q_min = plan->tiling == LITEVAR_TILING_PATCH ? 1 : (auto_patch ? 48 : 1 << 30);
    const int key_min = plan->tiling == LITEVAR_TILING_PATCH ? 4 : 32;
    st.q_patch = st.s_k >= q_min;
    st.first_patch = k0 + 1;
    if (st.q_patch) {  // patch key tiles only together with patch query tiles
      int first = 0;
      while (first <= k0 && sc.scale[first] < key_min) ++first;
      if (k0 + 1 - first > kMaxPatchScales) first = k0 + 1 - kMaxPatchScales;
      st.first_patch = first;
    }
    st.raster_len = sc.off[st.first_patch];
    st.n_raster_tiles = (st.raster_len + kBlockN - 1) / kBlockN;
    if (st.q_patch) {
      for (int r = 0; r < st.s_k; r += kPatchRows)
        for (int c = 0; c < st.s_k; c += kPatchCols) st.q_geom.push_back(TileGeom{k0, r, c, 0});
    } else {
      for (int q0 = 0; q0 < st.n_k; q0 += kBlockM) st.q_geom.push_back(TileGeom{-1, q0, 0, 0});
    }
    for (int t0 = 0; t0 < st.raster_len; t0 += kBlockN) st.key_geom.push_back(TileGeom{-1, t0, 0, 0});
    for (int j = st.first_patch; j <= k0; ++j)
      for (int r = 0; r < sc.scale[j]; r += kPatchRows)
        for (int c = 0; c < sc.scale[j]; c += kPatchCols) st.key_geom.push_back(TileGeom{j, r, c, j - st.first_patch});
    st.n_q_tiles = (int32_t)st.q_geom.size();
    st.n_key_tiles = (int32_t)st.key_geom.size();
    st.share = share && share->share_step && share->share_step[k0] != 0;
    st.sets.resize(n_sets);
  }

  // ---- device memory: the same sequence of take() calls sizes the blocks and then hands out the pointers
  std::vector<SetScratch> scratch((size_t)K * n_sets);
  SetTotals* d_totals = nullptr;
  int32_t* d_user = nullptr;
  Arena plan_mem, tmp_mem;
  auto lay_out = [&]() {
    plan->d_status = plan_mem.take<int32_t>(1);
    plan->d_radius = plan_mem.take<int32_t>((size_t)n_sets * K * K);
    plan->d_head_to_set = plan->head_to_set.empty() ? nullptr : plan_mem.take<int32_t>((size_t)n_heads);
    d_totals = tmp_mem.take<SetTotals>((size_t)K * n_sets);
    d_user = window->radius ? tmp_mem.take<int32_t>((size_t)n_sets * K * K) : nullptr;
    for (int k0 = 0; k0 < K; ++k0) {
      Step& st = plan->steps[k0];
      const size_t n_cand = (size_t)st.n_q_tiles * st.n_key_tiles;
      st.d_q_geom = plan_mem.take<TileGeom>(st.q_geom.size());
      st.d_key_geom = plan_mem.take<TileGeom>(st.key_geom.size());
      st.d_sets = plan_mem.take<SetDesc>((size_t)n_sets);
      for (int set = 0; set < n_sets; ++set) {
        StepSet& ss = st.sets[set];
        ss.d_bounds = plan_mem.take<int2>((size_t)(k0 + 1) * st.s_k);
        ss.d_row_ptr = plan_mem.take<int32_t>((size_t)st.n_q_tiles + 1);
        ss.d_order = plan_mem.take<int32_t>((size_t)(st.n_q_tiles + 1) / 2);
        ss.d_pairs = plan_mem.take<Pair>(n_cand);  // room for every candidate pair; n_pairs of them are used
        SetScratch& t = scratch[(size_t)k0 * n_sets + set];
        t.cls = tmp_mem.take<uint8_t>(n_cand);
        t.row_live = tmp_mem.take<int32_t>((size_t)st.n_k);
        t.partial_base = tmp_mem.take<int32_t>((size_t)st.n_q_tiles);
        t.blk = tmp_mem.take<int32_t>(n_cand);
      }
    }
  };
  lay_out();
  void *plan_block = nullptr, *tmp_block = nullptr;
  LV_TRY(cudaMalloc(&plan_block, plan_mem.used));
  plan->allocations.push_back(plan_block);
  LV_TRY(cudaMalloc(&tmp_block, tmp_mem.used));
  struct Free {
    void* p;
    ~Free() { cudaFree(p); }
  } free_tmp{tmp_block};
  plan_mem = Arena{static_cast<char*>(plan_block), 0};
  tmp_mem = Arena{static_cast<char*>(tmp_block), 0};
  lay_out();
  LV_TRY(cudaMemsetAsync(tmp_block, 0, tmp_mem.used, stream));  // counters, row_live, totals
  LV_TRY(cudaMemsetAsync(plan->d_status, 0, sizeof(int32_t), stream));

  // ---- A1: window tables on the device (default rule, or the caller's table normalised)
  if (window->radius)
    LV_TRY(cudaMemcpyAsync(d_user, window->radius, sizeof(int32_t) * n_sets * K * K, cudaMemcpyHostToDevice, stream));
  for (int set = 0; set < n_sets; ++set)
    window_table_kernel<<<1, 256, 0, stream>>>(sc, plan->shape, plan->n_global, plan->rho_num, plan->rho_den,
                                               d_user ? d_user + (size_t)set * K * K : nullptr,
                                               plan->d_radius + (size_t)set * K * K);
  plan->radius.resize((size_t)n_sets * K * K);
  LV_TRY(cudaMemcpyAsync(plan->radius.data(), plan->d_radius, sizeof(int32_t) * plan->radius.size(),
                         cudaMemcpyDeviceToHost, stream));
  if (plan->d_head_to_set)
    LV_TRY(cudaMemcpyAsync(plan->d_head_to_set, plan->head_to_set.data(), sizeof(int32_t) * n_heads,
                           cudaMemcpyHostToDevice, stream));

  // ---- A2 + A3, counting pass: bounds, classification of every candidate pair, per-tile counts and offsets
  for (int k0 = 0; k0 < K; ++k0) {
    Step& st = plan->steps[k0];
    LV_TRY(cudaMemcpyAsync(st.d_q_geom, st.q_geom.data(), sizeof(TileGeom) * st.q_geom.size(), cudaMemcpyHostToDevice,
                           stream));
    LV_TRY(cudaMemcpyAsync(st.d_key_geom, st.key_geom.data(), sizeof(TileGeom) * st.key_geom.size(),
                           cudaMemcpyHostToDevice, stream));
    const PlanGeom g{k0, st.s_k, st.n_k, st.L_k, st.n_key_tiles, plan->shape, st.raster_len, st.d_q_geom, st.d_key_geom};
    const dim3 grid2((unsigned)st.n_key_tiles, (unsigned)st.n_q_tiles);
    const int threads = st.n_q_tiles < 32 ? 32 : (st.n_q_tiles > 512 ? 512 : ((st.n_q_tiles + 31) / 32) * 32);
    for (int set = 0; set < n_sets; ++set) {
      StepSet& ss = st.sets[set];
      const SetScratch& t = scratch[(size_t)k0 * n_sets + set];
      SetTotals* tot = d_totals + (size_t)k0 * n_sets + set;
      const int32_t* d_radius_row = plan->d_radius + ((size_t)set * K + k0) * K;
      bounds_kernel<<<(unsigned)(((k0 + 1) * st.s_k + 255) / 256), 256, 0, stream>>>(sc, k0, d_radius_row, ss.d_bounds);
      classify_kernel<<<grid2, 128, 0, stream>>>(sc, g, ss.d_bounds, d_radius_row, t.cls, t.row_live, &tot->live_entries);
      empty_row_kernel<<<(unsigned)((st.n_k + 255) / 256), 256, 0, stream>>>(st.n_k, t.row_live, &tot->empty_row);
      count_scan_kernel<<<1, threads, 2 * sizeof(int32_t) * st.n_q_tiles, stream>>>(
          st.n_q_tiles, st.n_key_tiles, t.cls, ss.d_row_ptr, t.partial_base, &tot->n_pairs);
    }
  }
  std::vector<SetTotals> totals((size_t)K * n_sets);
  LV_TRY(cudaMemcpyAsync(totals.data(), d_totals, sizeof(SetTotals) * totals.size(), cudaMemcpyDeviceToHost, stream));
  LV_TRY(cudaGetLastError());
  LV_TRY(cudaStreamSynchronize(stream));
  size_t mask_rows = 0;
  for (int k0 = 0; k0 < K; ++k0)
    for (int set = 0; set < n_sets; ++set) {
      const SetTotals& t = totals[(size_t)k0 * n_sets + set];
      if (t.empty_row != 0) return LITEVAR_ERR_EMPTY_ROW;
      StepSet& ss = plan->steps[k0].sets[set];
      ss.n_pairs = t.n_pairs;
      ss.n_partial = t.n_partial;
      ss.n_full = t.n_full;
      ss.live_entries = (int64_t)t.live_entries;
      mask_rows += (size_t)t.n_partial * kBlockM;
    }

  // ---- A3, second pass: compaction in canonical order, element masks of the partial pairs, launch order
  void* mask_block = nullptr;
  LV_TRY(cudaMalloc(&mask_block, (mask_rows ? mask_rows : 1) * sizeof(uint4)));
  plan->allocations.push_back(mask_block);
  uint4* next_mask = static_cast<uint4*>(mask_block);
  std::vector<SetDesc> descs((size_t)K * n_sets);
  for (int k0 = 0; k0 < K; ++k0) {
    Step& st = plan->steps[k0];
    const PlanGeom g{k0, st.s_k, st.n_k, st.L_k, st.n_key_tiles, plan->shape, st.raster_len, st.d_q_geom, st.d_key_geom};
    const dim3 grid2((unsigned)st.n_key_tiles, (unsigned)st.n_q_tiles);
    for (int set = 0; set < n_sets; ++set) {
      StepSet& ss = st.sets[set];
      const SetScratch& t = scratch[(size_t)k0 * n_sets + set];
      SetTotals* tot = d_totals + (size_t)k0 * n_sets + set;
      const int32_t* d_radius_row = plan->d_radius + ((size_t)set * K + k0) * K;
      ss.d_mask = next_mask;
      next_mask += (size_t)ss.n_partial * kBlockM;
      compact_kernel<<<(unsigned)((st.n_q_tiles + 127) / 128), 128, 0, stream>>>(
          st.n_q_tiles, st.n_key_tiles, t.cls, ss.d_row_ptr, t.partial_base, ss.d_pairs, t.blk);
      mask_bits_kernel<<<grid2, 128, 0, stream>>>(sc, g, ss.d_bounds, d_radius_row, t.blk, ss.d_mask);
      launch_order_kernel<<<(unsigned)(((st.n_q_tiles + 1) / 2 + 127) / 128), 128, 0, stream>>>(st.n_q_tiles,
                                                                                             ss.d_row_ptr, ss.d_order);
      first_tile_kernel<<<(unsigned)((st.n_q_tiles + 127) / 128), 128, 0, stream>>>(st.n_q_tiles, ss.d_row_ptr,
                                                                                    ss.d_pairs, &tot->first_not_zero);
      if (small_step_candidate(st.n_q_tiles, st.n_key_tiles, !st.q_patch && st.first_patch == k0 + 1) &&
          ss.n_pairs >= 1 && ss.n_pairs <= 2)
        copy_first_pairs_kernel<<<1, 32, 0, stream>>>(ss.d_pairs, &tot->n_pairs, tot->first_pairs);
      descs[(size_t)k0 * n_sets + set] = SetDesc{ss.d_row_ptr, ss.d_pairs, ss.d_mask};
    }
    LV_TRY(cudaMemcpyAsync(st.d_sets, &descs[(size_t)k0 * n_sets], sizeof(SetDesc) * n_sets, cudaMemcpyHostToDevice,
                           stream));
  }
  LV_TRY(cudaMemcpyAsync(totals.data(), d_totals, sizeof(SetTotals) * totals.size(), cudaMemcpyDeviceToHost, stream));
  LV_TRY(cudaGetLastError());
  LV_TRY(cudaStreamSynchronize(stream));  // the scratch block is freed on return
  for (int k0 = 0; k0 < K; ++k0) {
    Step& st = plan->steps[k0];
    for (int set = 0; set < n_sets; ++set) {
      const SetTotals& t = totals[(size_t)k0 * n_sets + set];
      StepSet& ss = st.sets[set];
      ss.first_tile_zero = t.first_not_zero == 0;
      if (small_step_candidate(st.n_q_tiles, st.n_key_tiles, !st.q_patch && st.first_patch == k0 + 1) &&
          ss.n_pairs >= 1 && ss.n_pairs <= 2) {
        ss.small.n = ss.n_pairs;
        ss.small.pr[0] = t.first_pairs[0];
        ss.small.pr[1] = t.first_pairs[1];
      }
    }
  }
  return LITEVAR_OK;
}

// Which of the two tcgen05 kernels runs a step that is not a small one.  The kernel with one softmax thread per
// query row pays off on long tile lists (measured on B200: 5 to 8 % faster from about eight key tiles per query
// tile on, i.e. the last steps of the 512px schedule and the 2K step; 5 % slower on the two-to-six-tile lists of
// the 256px schedule, where the set-up of its longer pipeline is not written off).
bool use_row_kernel(const litevar_plan_t* plan, const Step& st) {
  if (plan->kernel == LITEVAR_KERNEL_TCGEN05_WS) return true;
  if (plan->kernel != LITEVAR_KERNEL_AUTO) return false;
  return (st.sets[0].n_pairs + st.n_q_tiles - 1) / st.n_q_tiles >= 8;
}

}  // namespace

extern "C" {

const char* litevar_status_string(litevar_status_t status) {
  switch (status) {
    case LITEVAR_OK: return "ok";
    case LITEVAR_ERR_INVALID_ARG: return "invalid argument";
    case LITEVAR_ERR_UNSUPPORTED: return "unsupported";
    case LITEVAR_ERR_EMPTY_ROW: return "window table leaves a query with no live key";
    case LITEVAR_ERR_ARCH: return "device is not compute capability 10.x";
    case LITEVAR_ERR_OOM: return "out of memory";
    case LITEVAR_ERR_CUDA: return "CUDA error";
    case LITEVAR_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

void litevar_plan_destroy(litevar_plan_t* plan) {
  if (!plan) return;
  for (void* p : plan->allocations) cudaFree(p);
  delete plan;
}

litevar_status_t litevar_attn_plan(const int32_t* scales, int32_t n_scales, int32_t n_heads, int32_t head_dim,
                                   float sm_scale, const litevar_window_t* window,
                                   const litevar_cfg_share_t* share, void* stream_, litevar_plan_t** out_plan) {
  if (!scales || !window || !out_plan) return LITEVAR_ERR_INVALID_ARG;
  if (n_scales < 1 || n_scales > kMaxScales || n_heads < 1 || head_dim < 1) return LITEVAR_ERR_INVALID_ARG;
  for (int i = 0; i < n_scales; ++i)
    if (scales[i] < 1 || scales[i] > kMaxScale) return LITEVAR_ERR_INVALID_ARG;
  if (window->shape != LITEVAR_WINDOW_SQUARE && window->shape != LITEVAR_WINDOW_BAND) return LITEVAR_ERR_INVALID_ARG;
  if (window->n_sets < 1 || window->n_sets > 64) return LITEVAR_ERR_INVALID_ARG;
  if (window->tiling < LITEVAR_TILING_AUTO || window->tiling > LITEVAR_TILING_PATCH) return LITEVAR_ERR_INVALID_ARG;
  if (!window->radius && (window->rho_den <= 0 || window->rho_num < 0 || window->n_global_scales < 0))
    return LITEVAR_ERR_INVALID_ARG;
  if (!window->radius && window->n_sets != 1) return LITEVAR_ERR_INVALID_ARG;
  if (window->head_to_set)
    for (int h = 0; h < n_heads; ++h)
      if (window->head_to_set[h] < 0 || window->head_to_set[h] >= window->n_sets) return LITEVAR_ERR_INVALID_ARG;
  if (head_dim != kHeadDim) return LITEVAR_ERR_UNSUPPORTED;

  int dev = 0;
  cudaDeviceProp prop;
  LV_CUDA(cudaGetDevice(&dev));
  LV_CUDA(cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10) return LITEVAR_ERR_ARCH;

  litevar_plan* plan = new (std::nothrow) litevar_plan();
  if (!plan) return LITEVAR_ERR_OOM;
  litevar_status_t result = LITEVAR_ERR_OOM;
  try {
    result = build_plan(plan, scales, n_scales, n_heads, sm_scale, window, share, dev, prop.multiProcessorCount,
                        static_cast<cudaStream_t>(stream_));
  } catch (...) {  // a host container ran out of memory: nothing crosses the C boundary
    result = LITEVAR_ERR_OOM;
  }
  if (result != LITEVAR_OK) {
    (void)cudaStreamSynchronize(static_cast<cudaStream_t>(stream_));  // planner kernels may still use the buffers
    litevar_plan_destroy(plan);
    return result;
  }
  *out_plan = plan;
  return LITEVAR_OK;
}

// Launch parameters of a step that do not depend on the tensors.
static void fill_step_params(const litevar_plan_t* plan, const Step& st, int32_t step_k, int32_t batch_pairs,
                             FwdParams& p) {
  memset(&p, 0, sizeof(p));
  p.sets = st.d_sets;
  p.head_to_set = plan->n_sets > 1 ? plan->d_head_to_set : nullptr;
  p.set0 = SetDesc{st.sets[0].d_row_ptr, st.sets[0].d_pairs, st.sets[0].d_mask};
  p.order = st.sets[0].d_order;
  p.n_k = st.n_k;
  p.L_k = st.L_k;
  p.n_heads = plan->n_heads;
  p.q_geom = st.d_q_geom;
  p.key_geom = st.d_key_geom;
  p.s_k = st.s_k;
  p.q_patch = st.q_patch ? 1 : 0;
  p.raster_len = st.raster_len;
  p.first_patch = st.first_patch;
  p.n_patch_scales = step_k - st.first_patch;
  for (int i = 0; i < kMaxPatchScales; ++i) {
    const int j = st.first_patch + i;
    p.patch_scale[i] = j < step_k ? plan->sched.scale[j] : 0;
    p.patch_off[i] = j < step_k ? plan->sched.off[j] : 0;
  }
  p.batch_computed = st.share ? batch_pairs : 2 * batch_pairs;
  p.share_offset = st.share ? batch_pairs : 0;
  p.sm_scale = plan->sm_scale;
  p.status = plan->d_status;
  p.overlap_launch = 1;
  p.first_tile_zero = st.raster_len > 0 ? 1 : 0;  // key tile 0 must be the raster tile of cache rows [0, 128)
  for (const StepSet& ss : st.sets) p.first_tile_zero &= ss.first_tile_zero ? 1 : 0;
  p.pairs_per_tile = (st.sets[0].n_pairs + st.n_q_tiles - 1) / st.n_q_tiles;
  p.units_per_group = units_per_l2_group(st.L_k, p.n_heads * p.batch_computed);
}

litevar_status_t litevar_attn_forward(const litevar_plan_t* plan, int32_t step_k, int32_t batch_pairs,
                                      const void* Q, const litevar_strides_t* sq, const void* Kc,
                                      const litevar_strides_t* sk, const void* Vc, const litevar_strides_t* sv,
                                      void* out, const litevar_strides_t* so, void* stream_) {
  if (!plan || !Q || !Kc || !Vc || !out) return LITEVAR_ERR_INVALID_ARG;
  if (step_k < 1 || step_k > plan->sched.n_scales || batch_pairs < 1) return LITEVAR_ERR_INVALID_ARG;
  if (!strides_ok(sq) || !strides_ok(sk) || !strides_ok(sv) || !strides_ok(so)) return LITEVAR_ERR_INVALID_ARG;
  if (((uintptr_t)Q | (uintptr_t)Kc | (uintptr_t)Vc | (uintptr_t)out) & 15) return LITEVAR_ERR_INVALID_ARG;
  if (!on_plan_device(plan)) return LITEVAR_ERR_INVALID_ARG;
  const Step& st = plan->steps[step_k - 1];
  FwdParams p;
  fill_step_params(plan, st, step_k, batch_pairs, p);
  p.q = static_cast<const uint16_t*>(Q);
  p.k = static_cast<const uint16_t*>(Kc);
  p.v = static_cast<const uint16_t*>(Vc);
  p.out = static_cast<uint16_t*>(out);
  p.q_sb = sq->batch; p.q_sh = sq->head; p.q_st = sq->token;
  p.k_sb = sk->batch; p.k_sh = sk->head; p.k_st = sk->token;
  p.v_sb = sv->batch; p.v_sh = sv->head; p.v_st = sv->token;
  p.o_sb = so->batch; p.o_sh = so->head; p.o_st = so->token;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (const int mode = small_mode(plan, st, (long long)p.n_heads * p.batch_computed)) {
    if (launch_forward_small(p, st.sets[0].small, mode, plan->n_sm, stream) != cudaSuccess) {
      (void)cudaGetLastError();
      return LITEVAR_ERR_CUDA;
    }
    return LITEVAR_OK;
  }
  if (plan->kernel == LITEVAR_KERNEL_SIMT) {
    cudaError_t e = launch_forward_simt(p, st.n_q_tiles, stream);
    if (e != cudaSuccess) {
      (void)cudaGetLastError();
      return LITEVAR_ERR_CUDA;
    }
    return LITEVAR_OK;
  }
  if (use_row_kernel(plan, st)) return launch_forward_ws(p, st.n_q_tiles, stream);
  return launch_forward_tcgen05(p, st.n_q_tiles, stream);
}

litevar_status_t litevar_attn_forward_kv8(const litevar_plan_t* plan, int32_t step_k, int32_t batch_pairs,
                                          const void* Q, const litevar_strides_t* sq, const int8_t* Kcodes,
                                          const float* Kscale, const float* Kzero, const int8_t* Vcodes,
                                          const float* Vscale, const float* Vzero, const litevar_strides_t* scodes,
                                          const litevar_strides_t* srow, void* out, const litevar_strides_t* so,
                                          void* stream_) {
  if (!plan || !Q || !Kcodes || !Kscale || !Kzero || !Vcodes || !Vscale || !Vzero || !out || !scodes || !srow)
    return LITEVAR_ERR_INVALID_ARG;
  if (step_k < 1 || step_k > plan->sched.n_scales || batch_pairs < 1) return LITEVAR_ERR_INVALID_ARG;
  if (!strides_ok(sq) || !strides_ok(so)) return LITEVAR_ERR_INVALID_ARG;
  if (scodes->batch < 0 || scodes->head < 0 || scodes->token < kHeadDim || (scodes->batch | scodes->head | scodes->token) & 15)
    return LITEVAR_ERR_INVALID_ARG;  // every code row starts on a 16-byte boundary
  if (srow->batch < 0 || srow->head < 0 || srow->token != 1) return LITEVAR_ERR_INVALID_ARG;
  if (((uintptr_t)Q | (uintptr_t)Kcodes | (uintptr_t)Vcodes | (uintptr_t)out) & 15) return LITEVAR_ERR_INVALID_ARG;
  if (((uintptr_t)Kscale | (uintptr_t)Kzero | (uintptr_t)Vscale | (uintptr_t)Vzero) & 3) return LITEVAR_ERR_INVALID_ARG;
  if (!on_plan_device(plan)) return LITEVAR_ERR_INVALID_ARG;
  const Step& st = plan->steps[step_k - 1];
  if (st.q_patch || st.first_patch != step_k) return LITEVAR_ERR_UNSUPPORTED;  // raster tiles only
  FwdParams p;
  fill_step_params(plan, st, step_k, batch_pairs, p);
  p.q = static_cast<const uint16_t*>(Q);
  p.out = static_cast<uint16_t*>(out);
  p.q_sb = sq->batch; p.q_sh = sq->head; p.q_st = sq->token;
  p.o_sb = so->batch; p.o_sh = so->head; p.o_st = so->token;
  p.k8 = Kcodes; p.v8 = Vcodes;
  p.k_scale = Kscale; p.k_zero = Kzero; p.v_scale = Vscale; p.v_zero = Vzero;
  p.c_sb = scodes->batch; p.c_sh = scodes->head; p.c_st = scodes->token;
  p.z_sb = srow->batch; p.z_sh = srow->head;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (const int mode = small_mode(plan, st, (long long)p.n_heads * p.batch_computed)) {
    if (launch_forward_small_kv8(p, st.sets[0].small, mode, plan->n_sm, stream) != cudaSuccess) {
      (void)cudaGetLastError();
      return LITEVAR_ERR_CUDA;
    }
    return LITEVAR_OK;
  }
  return launch_forward_tcgen05_kv8(p, st.n_q_tiles, stream);
}

static litevar_status_t check_step_set(const litevar_plan_t* plan, int32_t step_k, int32_t set) {
  if (!plan || step_k < 1 || step_k > plan->sched.n_scales || set < 0 || set >= plan->n_sets)
    return LITEVAR_ERR_INVALID_ARG;
  return LITEVAR_OK;
}

litevar_status_t litevar_plan_stats(const litevar_plan_t* plan, int32_t step_k, int32_t set, int64_t* live_entries,
                                    int64_t* live_tiles, int64_t* full_tiles, int64_t* partial_tiles) {
  litevar_status_t s = check_step_set(plan, step_k, set);
  if (s != LITEVAR_OK) return s;
  const StepSet& ss = plan->steps[step_k - 1].sets[set];
  if (live_entries) *live_entries = ss.live_entries;
  if (live_tiles) *live_tiles = ss.n_pairs;
  if (full_tiles) *full_tiles = ss.n_full;
  if (partial_tiles) *partial_tiles = ss.n_partial;
  return LITEVAR_OK;
}

litevar_status_t litevar_plan_tile_counts(const litevar_plan_t* plan, int32_t step_k, int32_t set,
                                          int32_t* n_q_tiles, int32_t* n_key_tiles, int32_t* n_pairs) {
  litevar_status_t s = check_step_set(plan, step_k, set);
  if (s != LITEVAR_OK) return s;
  const Step& st = plan->steps[step_k - 1];
  if (n_q_tiles) *n_q_tiles = st.n_q_tiles;
  if (n_key_tiles) *n_key_tiles = st.n_key_tiles;
  if (n_pairs) *n_pairs = st.sets[set].n_pairs;
  return LITEVAR_OK;
}

litevar_status_t litevar_plan_export_tiles(const litevar_plan_t* plan, int32_t step_k, int32_t set,
                                           int32_t* q_tile_geom, int32_t* key_tile_geom, int32_t* row_ptr,
                                           int32_t* pair_key_tile, uint8_t* pair_is_full) {
  litevar_status_t s = check_step_set(plan, step_k, set);
  if (s != LITEVAR_OK) return s;
  if (!on_plan_device(plan)) return LITEVAR_ERR_INVALID_ARG;
  const Step& st = plan->steps[step_k - 1];
  const StepSet& ss = st.sets[set];
  auto put = [&](int32_t* out, const TileGeom& g, int side, int base, int limit) {
    if (g.scale < 0) {  // raster: one row of up to 128 consecutive tokens
      int valid = limit - g.a < kBlockM ? limit - g.a : kBlockM;
      out[0] = g.a; out[1] = kBlockM; out[2] = 0; out[3] = 1; out[4] = valid;
    } else {            // patch: kPatchRows x kPatchCols cells at (a, b), clipped to the grid
      int vr = side - g.a < kPatchRows ? side - g.a : kPatchRows;
      int vc = side - g.b < kPatchCols ? side - g.b : kPatchCols;
      out[0] = base + g.a * side + g.b; out[1] = kPatchCols; out[2] = side; out[3] = vr; out[4] = vc;
    }
  };
  if (q_tile_geom)
    for (int i = 0; i < st.n_q_tiles; ++i) put(q_tile_geom + 5 * i, st.q_geom[i], st.s_k, 0, st.n_k);
  if (key_tile_geom)
    for (int i = 0; i < st.n_key_tiles; ++i) {
      const TileGeom& g = st.key_geom[i];
      const int side = g.scale < 0 ? 0 : plan->sched.scale[g.scale];
      const int base = g.scale < 0 ? 0 : plan->sched.off[g.scale];
      put(key_tile_geom + 5 * i, g, side, base, st.raster_len);
    }
  LV_CUDA(cudaDeviceSynchronize());
  if (row_ptr)
    LV_CUDA(cudaMemcpy(row_ptr, ss.d_row_ptr, sizeof(int32_t) * (st.n_q_tiles + 1), cudaMemcpyDeviceToHost));
  if ((pair_key_tile || pair_is_full) && ss.n_pairs > 0) {
    std::vector<Pair> pairs(ss.n_pairs);
    LV_CUDA(cudaMemcpy(pairs.data(), ss.d_pairs, sizeof(Pair) * ss.n_pairs, cudaMemcpyDeviceToHost));
    for (int i = 0; i < ss.n_pairs; ++i) {
      if (pair_key_tile) pair_key_tile[i] = pairs[i].key_tile;
      if (pair_is_full) pair_is_full[i] = pairs[i].mask_block < 0 ? 1 : 0;
    }
  }
  return LITEVAR_OK;
}

litevar_status_t litevar_plan_export_bounds(const litevar_plan_t* plan, int32_t step_k, int32_t set,
                                            int32_t* radius, int32_t* bounds) {
  litevar_status_t s = check_step_set(plan, step_k, set);
  if (s != LITEVAR_OK) return s;
  const int K = plan->sched.n_scales;
  const Step& st = plan->steps[step_k - 1];
  if (radius)
    memcpy(radius, plan->radius.data() + ((size_t)set * K + (step_k - 1)) * K, sizeof(int32_t) * K);
  if (bounds) {
    if (!on_plan_device(plan)) return LITEVAR_ERR_INVALID_ARG;
    LV_CUDA(cudaDeviceSynchronize());
    LV_CUDA(cudaMemcpy(bounds, st.sets[set].d_bounds, sizeof(int2) * step_k * st.s_k, cudaMemcpyDeviceToHost));
  }
  return LITEVAR_OK;
}

litevar_status_t litevar_plan_materialize_mask(const litevar_plan_t* plan, int32_t step_k, int32_t set,
                                               void* dev_bits, void* stream_) {
  litevar_status_t s = check_step_set(plan, step_k, set);
  if (s != LITEVAR_OK) return s;
  if (!dev_bits || !on_plan_device(plan)) return LITEVAR_ERR_INVALID_ARG;
  const Step& st = plan->steps[step_k - 1];
  const StepSet& ss = st.sets[set];
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  size_t words = (size_t)((st.L_k + 31) / 32);
  LV_CUDA(cudaMemsetAsync(dev_bits, 0, sizeof(uint32_t) * words * st.n_k, stream));
  SetDesc sd{ss.d_row_ptr, ss.d_pairs, ss.d_mask};
  PlanGeom g{step_k - 1, st.s_k, st.n_k, st.L_k, st.n_key_tiles, plan->shape, st.raster_len, st.d_q_geom, st.d_key_geom};
  materialize_kernel<<<(unsigned)st.n_q_tiles, 128, 0, stream>>>(sd, plan->sched, g, static_cast<uint32_t*>(dev_bits));
  LV_CUDA(cudaGetLastError());
  return LITEVAR_OK;
}

litevar_status_t litevar_plan_poll_device_status(const litevar_plan_t* plan) {
  if (!plan || !on_plan_device(plan)) return LITEVAR_ERR_INVALID_ARG;
  int32_t v = 0;
  LV_CUDA(cudaDeviceSynchronize());
  LV_CUDA(cudaMemcpy(&v, plan->d_status, sizeof(v), cudaMemcpyDeviceToHost));
  if (v != 0) {
    LV_CUDA(cudaMemset(plan->d_status, 0, sizeof(v)));
    return LITEVAR_ERR_DEVICE_TIMEOUT;
  }
  return LITEVAR_OK;
}

litevar_status_t litevar_plan_set_kernel(litevar_plan_t* plan, int32_t kernel) {
  if (!plan || kernel < LITEVAR_KERNEL_AUTO || kernel > LITEVAR_KERNEL_TCGEN05_WS || kernel == LITEVAR_KERNEL_SMALL) return LITEVAR_ERR_INVALID_ARG;
  plan->kernel = kernel;
  return LITEVAR_OK;
}

litevar_status_t litevar_plan_step_kernel(const litevar_plan_t* plan, int32_t step_k, int32_t batch_pairs,
                                          int32_t* kernel) {
  if (!plan || !kernel || step_k < 1 || step_k > plan->sched.n_scales || batch_pairs < 1) return LITEVAR_ERR_INVALID_ARG;
  const Step& st = plan->steps[step_k - 1];
  const long long units = (long long)plan->n_heads * (st.share ? batch_pairs : 2 * batch_pairs);
  *kernel = plan->kernel == LITEVAR_KERNEL_SIMT ? LITEVAR_KERNEL_SIMT
            : small_mode(plan, st, units)       ? LITEVAR_KERNEL_SMALL
            : use_row_kernel(plan, st)          ? LITEVAR_KERNEL_TCGEN05_WS
                                                : LITEVAR_KERNEL_TCGEN05;
  return LITEVAR_OK;
}

}  // extern "C"
