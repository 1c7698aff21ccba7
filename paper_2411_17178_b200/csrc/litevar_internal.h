// Internal definitions shared by the translation units of liblitevar (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "litevar.h"

namespace litevar {

constexpr int kMaxScales = 16;
constexpr int kMaxScale = 256;
constexpr int kHeadDim = 64;
constexpr int kBlockM = 128;  // query slots per tile
constexpr int kBlockN = 128;  // key slots per tile
constexpr int kMaskWordsPerRow = kBlockN / 32;

// Schedule of one plan, passed to kernels by value (paper Section 2: n_k = s_k^2, off_j, L_k).
struct Schedule {
  int32_t n_scales;
  int32_t scale[kMaxScales];
  int32_t off[kMaxScales + 1];  // off[j] = tokens before scale j+1 (0-based j); off[K] = total
};

// One live (query tile, key tile) pair: key tile index and index of its 128x128-bit mask block
// (-1: every slot pair is live, no element mask).
struct Pair {
  int32_t key_tile;
  int32_t mask_block;
};

// Geometry of one query or key tile (128 slots).  Raster: scale < 0, slot m is token a + m (query tiles:
// token of the current scale; key tiles: cache row, valid below the end of the raster prefix).  Patch:
// scale = 0-based scale index, slot m is grid cell (a + m / kPatchCols, b + m % kPatchCols) of that scale.
struct TileGeom {
  int32_t scale, a, b, map_slot;  // map_slot: index of the scale's tensor maps in the forward kernel (patch tiles)
};
constexpr int kPatchRows = 8, kPatchCols = 16;  // kPatchRows * kPatchCols == 128
constexpr int kMaxPatchScales = 8;              // key scales that can be tiled in 2-D patches

// The whole tile list of a step with one query tile and at most two key tiles, passed to the small-step
// kernel by value (saves it two dependent global loads).
struct SmallLists {
  int32_t n;
  Pair pr[2];
};

// Device-visible tile plan of one (step, window set).
struct SetDesc {
  const int32_t* row_ptr;  // [n_q_tiles + 1]
  const Pair* pairs;       // [n_pairs]
  const uint4* mask;       // [n_partial][kBlockM] : 128 key bits per query slot
};

struct StepSet {
  int32_t n_pairs = 0, n_partial = 0, n_full = 0;
  int64_t live_entries = 0;
  int32_t* d_row_ptr = nullptr;
  Pair* d_pairs = nullptr;
  uint4* d_mask = nullptr;
  int2* d_bounds = nullptr;  // [k][s_k] {lo, hi} per key scale and query row/column (SQUARE)
  bool first_tile_zero = false;  // every query tile lists key tile 0 first
  int32_t* d_order = nullptr;  // [ceil(n_q_tiles / 2)] query-tile pairs, heaviest first
  SmallLists small = {-1, {{0, 0}, {0, 0}}};  // host copy of the tile list of a small step (n < 0: not a small step)
};

struct Step {
  int32_t s_k = 0, n_k = 0, L_k = 0, n_q_tiles = 0, n_key_tiles = 0;
  bool share = false;
  bool q_patch = false;       // query tiles are 2-D patches of the current scale's grid
  int32_t first_patch = 0;    // key scales with 0-based index >= first_patch are tiled in patches (== step count: none)
  int32_t raster_len = 0;     // cache rows [0, raster_len) are covered by raster key tiles
  int32_t n_raster_tiles = 0;
  litevar::TileGeom* d_q_geom = nullptr;    // [n_q_tiles]
  litevar::TileGeom* d_key_geom = nullptr;  // [n_key_tiles]
  std::vector<litevar::TileGeom> q_geom, key_geom;  // host copies
  std::vector<StepSet> sets;
  SetDesc* d_sets = nullptr;  // [n_sets]
};

// Arguments of one forward launch, common to both kernels.
struct FwdParams {
  const SetDesc* sets;          // [n_sets] for this step
  const int32_t* head_to_set;   // [H] or nullptr (all heads use set 0)
  SetDesc set0;                 // copy of sets[0]: saves the kernels one dependent load when there is one set
  const int32_t* order;         // launch order of the query-tile pairs (heaviest first), or nullptr: natural order
  const uint16_t* q;
  const uint16_t* k;
  const uint16_t* v;
  uint16_t* out;
  int64_t q_sb, q_sh, q_st;     // element strides: batch, head, token
  int64_t k_sb, k_sh, k_st;
  int64_t v_sb, v_sh, v_st;
  int64_t o_sb, o_sh, o_st;
  int32_t n_k, L_k, n_heads;
  // tile geometry; q_geom == nullptr: raster tiles everywhere (tile i = tokens [128 i, 128 i + 128))
  const TileGeom* q_geom;
  const TileGeom* key_geom;
  int32_t s_k;              // side of the current scale's grid
  int32_t q_patch;          // query tiles are patches (host: rank of the Q and output tensor maps)
  int32_t raster_len;       // cache rows covered by raster key tiles (L_k when there are no patch tiles)
  int32_t first_patch;      // first key scale (0-based) tiled in patches
  int32_t n_patch_scales;   // number of such scales (<= kMaxPatchScales)
  int32_t patch_scale[kMaxPatchScales];  // their grid sides
  int32_t patch_off[kMaxPatchScales];    // their first cache rows
  int32_t batch_computed;       // rows the grid covers (B when shared, else 2B)
  int32_t share_offset;         // B when the step is shared (second store at row b + B), else 0
  float sm_scale;
  int32_t* status;              // device word, set non-zero when a bounded wait expires
  int32_t pairs_per_tile;       // average live key tiles per query tile (0: unknown); picks the kernel build
  int32_t first_tile_zero;      // 1: every query tile's list starts with key tile 0 (its copies start at once)
  // 8-bit K/V cache (litevar_attn_forward_kv8): int8 codes [2B, H, rows, 64] with byte strides c_*, and one fp32
  // scale and zero point per row, [2B, H, rows] with strides z_sb, z_sh (rows contiguous); k and v are unused
  const int8_t* k8;
  const int8_t* v8;
  const float *k_scale, *k_zero, *v_scale, *v_zero;
  int64_t c_sb, c_sh, c_st, z_sb, z_sh;
  int32_t units_per_group;      // launch order of the tensor-core kernels: (batch row, head) units per L2 group
  int32_t overlap_launch;       // 1: the tensor-core kernel may start its set-up before the previous kernel of the
                                // stream has finished (the plan it reads was complete long before)
};

// SM count of the current device, looked up once per device (the attribute query costs a microsecond).
// L2 size of the current device in bytes, looked up once per device.
inline long long current_l2_bytes() {
  static long long cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 64ll << 20;
  long long n = cached[dev];
  if (n == 0) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrL2CacheSize, dev) != cudaSuccess || v <= 0) return 64ll << 20;
    cached[dev] = n = v;  // benign race: every writer stores the same value
  }
  return n;
}

inline int current_sm_count() {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  int n = cached[dev];
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    cached[dev] = n;  // benign race: every writer stores the same value
  }
  return n;
}

// (batch row, head) units whose K and V prefixes (L_k rows of 128 B each) together fill half of L2: the group size
// of the tensor-core kernels' launch order.
inline int units_per_l2_group(int L_k, int n_units) {
  const long long per_unit = 2ll * L_k * kHeadDim * 2;
  long long g = (current_l2_bytes() / 2) / (per_unit > 0 ? per_unit : 1);
  if (g < 1) g = 1;
  if (g > n_units) g = n_units;
  return (int)g;
}

cudaError_t launch_forward_simt(const FwdParams& p, int n_q_tiles, cudaStream_t stream);

// Small steps (one query tile, at most two raster key tiles): warp-level mma on a shared-memory copy of the whole
// K/V prefix.  `small_step_candidate` is the plan-time test; `small_step_mode` decides per launch from the
// work and the number of (batch row, head) units: 0 = use the tcgen05 kernel, 1 = one warp per 16 query rows, 2 = two.
// `lists` is set 0's tile list (per-head sets are looked up on the device).
bool small_step_candidate(int n_q_tiles, int n_key_tiles, bool raster_only);
int small_step_mode(int n_k, int L_k, long long units, int n_sm);
cudaError_t launch_forward_small(const FwdParams& p, const SmallLists& lists, int mode, int n_sm, cudaStream_t stream);
// The same kernel reading an 8-bit K/V cache (p.k8 ...).
cudaError_t launch_forward_small_kv8(const FwdParams& p, const SmallLists& lists, int mode, int n_sm,
                                     cudaStream_t stream);

// Tensor-core path.  Returns LITEVAR_OK or an error status (tensor-map encoding can fail).
litevar_status_t launch_forward_tcgen05(const FwdParams& p, int n_q_tiles, cudaStream_t stream);
// The same kernel reading an 8-bit K/V cache (p.k8 ...; raster tiles only).
litevar_status_t launch_forward_tcgen05_kv8(const FwdParams& p, int n_q_tiles, cudaStream_t stream);
// The same path with one softmax thread per query row (register reallocation between warpgroups).
litevar_status_t launch_forward_ws(const FwdParams& p, int n_q_tiles, cudaStream_t stream);

#ifdef __CUDACC__
// 8-bit cache rows (paper Section 4): 16 int8 codes of one row -> 16 bf16 values code * s + z, as two 16-byte chunks.
// One fused multiply-add per pair and no integer conversion (that pipe is the exponential pipe): the codes are biased
// by 128 (one XOR per four); a byte permute puts each biased code u into the second byte of the bit pattern of 2^15,
// which is the fp32 number 32768 + u; and fma(32768 + u, s, z') with z' = z - 32896 s (shifted_zero, rounded once
// per row) is code * s + z up to the rounding of z': 2^-9 of a quantisation step s.
__device__ __forceinline__ float shifted_zero_point(float zero, float scale) { return fmaf(-32896.f, scale, zero); }
__device__ __forceinline__ void widen_codes16(const uint4& codes, float scale, float shifted_zero, uint4& lo, uint4& hi) {
  const float2 sc2 = make_float2(scale, scale), zs2 = make_float2(shifted_zero, shifted_zero);
  const uint32_t w[4] = {codes.x, codes.y, codes.z, codes.w};
  uint32_t o[8];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const uint32_t word = w[e] ^ 0x80808080u;
    uint32_t f[4];
    // prmt: selector nibbles 0-3 pick bytes of the first operand, 4-7 of the second
    asm("prmt.b32 %0, %1, %2, 0x7604;" : "=r"(f[0]) : "r"(word), "r"(0x47000000u));
    asm("prmt.b32 %0, %1, %2, 0x7614;" : "=r"(f[1]) : "r"(word), "r"(0x47000000u));
    asm("prmt.b32 %0, %1, %2, 0x7624;" : "=r"(f[2]) : "r"(word), "r"(0x47000000u));
    asm("prmt.b32 %0, %1, %2, 0x7634;" : "=r"(f[3]) : "r"(word), "r"(0x47000000u));
    const float2 x01 = __ffma2_rn(make_float2(__uint_as_float(f[0]), __uint_as_float(f[1])), sc2, zs2);
    const float2 x23 = __ffma2_rn(make_float2(__uint_as_float(f[2]), __uint_as_float(f[3])), sc2, zs2);
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o[2 * e]) : "f"(x01.y), "f"(x01.x));
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o[2 * e + 1]) : "f"(x23.y), "f"(x23.x));
  }
  lo = make_uint4(o[0], o[1], o[2], o[3]);
  hi = make_uint4(o[4], o[5], o[6], o[7]);
}
#endif

}  // namespace litevar

struct litevar_plan {
  litevar::Schedule sched;
  int32_t n_heads = 0, n_sets = 1, shape = 0, n_global = 0, rho_num = 1, rho_den = 4, tiling = 0;
  float sm_scale = 0.125f;
  int32_t kernel = LITEVAR_KERNEL_AUTO;
  int device = 0, n_sm = 148;
  std::vector<int32_t> radius;        // [n_sets][K][K]
  std::vector<int32_t> head_to_set;   // [H] (empty when n_sets == 1)
  int32_t* d_head_to_set = nullptr;
  int32_t* d_radius = nullptr;        // [n_sets][K][K]
  int32_t* d_status = nullptr;
  std::vector<litevar::Step> steps;   // [K]
  std::vector<void*> allocations;     // every cudaMalloc of the plan
};
