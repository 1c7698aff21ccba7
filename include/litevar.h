/*
 * litevar.h -- C ABI of the LiteVAR attention library for NVIDIA B200 (sm_100a).
 *
 * One operation: the attention that a VAR image generator runs at every coarse-to-fine
 * scale step (the current scale's queries against the K/V cache of all scales so far),
 * under LiteVAR's multi-diagonal window mask (MDWA, paper Section 2) and with LiteVAR's
 * attention sharing across classifier-free guidance (ASC, paper Section 3).  Beside it: the
 * window calibration of Section 2 on saved attention maps (litevar_calibrate_windows) and the
 * dynamic 8-bit quantiser of Q, K and V of Section 4 (litevar_quantize_rows, litevar_quantize_qkv).
 *
 * Notation (paper Section 2).  Scales s_1..s_K; scale k holds n_k = s_k^2 tokens in
 * row-major order of its s_k x s_k grid; off_j = sum_{i<j} n_i; L_k = sum_{i<=k} n_i.
 * Step k (1-based): queries are the n_k tokens of scale k, keys/values are rows
 * [0, L_k) of the cache, so the step-k attention map is [n_k, L_k].
 *
 * General rules.  No call throws, aborts or traps.  Every call returns a status; output
 * arguments are written only on LITEVAR_OK.  "host" / "device" below say where a pointer
 * must live.  Tensors passed to litevar_attn_forward are borrowed for the duration of the
 * asynchronous work; the plan owns everything it allocates.
 */
#ifndef LITEVAR_H_
#define LITEVAR_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct litevar_plan litevar_plan_t; /* opaque; owns its device buffers */

typedef enum {
  LITEVAR_OK = 0,
  LITEVAR_ERR_INVALID_ARG = 1,    /* NULL pointer, size or index out of range, misaligned tensor */
  LITEVAR_ERR_UNSUPPORTED = 2,    /* valid request that this library does not implement */
  LITEVAR_ERR_EMPTY_ROW = 3,      /* the window table leaves some query with no live key */
  LITEVAR_ERR_ARCH = 4,           /* current device is not compute capability 10.x */
  LITEVAR_ERR_OOM = 5,            /* device or host allocation failed */
  LITEVAR_ERR_CUDA = 6,           /* a CUDA runtime/driver call failed */
  LITEVAR_ERR_DEVICE_TIMEOUT = 7  /* a bounded device-side wait expired (see poll) */
} litevar_status_t;

/* Window shapes.  SQUARE: key (r',c') of scale j is live for query (r,c) of scale k iff
 * |r' - ctr_j(r)| <= w and |c' - ctr_j(c)| <= w with ctr_j(x) = floor((2x+1) s_j / (2 s_k)),
 * clipped at the grid border (the local window of paper Section 2 / Fig. 2(a), read as a 2-D
 * neighbourhood of the co-located key cell).  BAND: key token t' of scale j is live iff
 * |t' - floor((2q+1) n_j / (2 n_k))| <= w, the literal 1-D band about the part's diagonal in
 * the flattened attention map. */
enum { LITEVAR_WINDOW_SQUARE = 0, LITEVAR_WINDOW_BAND = 1 };

/* Tile geometry of the plan.  RASTER: every query and key tile is 128 consecutive tokens.  PATCH:
 * a query tile is an 8 x 16 patch of the current scale's grid and the keys of the larger scales
 * are tiled in 8 x 16 patches of their own grids (grid-aligned), so that a 2-D window leaves whole
 * tiles dead; the coarse scales in front stay raster.  AUTO picks PATCH for SQUARE windows at steps
 * whose grid side is at least 48 (key scales of side >= 32 in patches, at most 8 of them) and RASTER
 * otherwise. */
enum { LITEVAR_TILING_AUTO = 0, LITEVAR_TILING_RASTER = 1, LITEVAR_TILING_PATCH = 2 };

/* Window specification (paper Section 2: one window width per part of the step-k map; the
 * first parts stay global, "MDWA implementation details"). */
typedef struct {
  int32_t shape;            /* LITEVAR_WINDOW_SQUARE or LITEVAR_WINDOW_BAND */
  int32_t n_global_scales;  /* key scales j <= this are fully live (paper: the merged first part, 3) */
  int32_t rho_num, rho_den; /* default rule when radius == NULL: w_j = floor((2*num*s_j + den) / (2*den)),
                               i.e. rho * s_j rounded half up (SQUARE) or rho * n_j (BAND) */
  const int32_t* radius;    /* optional host table [n_sets][n_scales][n_scales], entry (set, k-1, j-1);
                               -1 = whole part live; copied at plan time; entries with j > k ignored */
  int32_t n_sets;           /* number of window tables (paper: widths are chosen per head); >= 1 */
  const int32_t* head_to_set; /* host [n_heads], values in [0, n_sets); NULL = all heads use set 0 */
  int32_t tiling;           /* LITEVAR_TILING_*; changes the tile lists and the speed, never the result */
} litevar_window_t;

/* CFG sharing (paper Section 3): at a shared step the unconditional half of the batch
 * receives a copy of the conditional half's attention output and is not computed. */
typedef struct {
  const uint8_t* share_step; /* host [n_scales], 1 = share at that step; NULL = never */
} litevar_cfg_share_t;

/* Element strides of a [2B, H, tokens, head_dim] tensor; head_dim has stride 1. */
typedef struct {
  int64_t batch, head, token;
} litevar_strides_t;

/* Forward kernel selection (testing / measurement). */
enum {
  LITEVAR_KERNEL_AUTO = 0,    /* per step: the small-step kernel where the step fits it, else a tcgen05 kernel (the one
                                 with a softmax thread per query row on long tile lists) */
  LITEVAR_KERNEL_SIMT = 1,    /* plain CUDA-core kernel (slow; cross-check and bring-up) */
  LITEVAR_KERNEL_TCGEN05 = 2, /* tcgen05/TMEM/TMA kernel with two softmax threads per query row, for every step */
  LITEVAR_KERNEL_SMALL = 3,   /* reported by litevar_plan_step_kernel only: warp-level mma kernel for steps with one
                                 query tile, at most two raster key tiles and little work */
  LITEVAR_KERNEL_TCGEN05_WS = 4 /* tcgen05 kernel with one softmax thread per query row, for every step */
};

/*
 * Build the per-step tile plan on the device (paper Section 2: parts, windows, global parts).
 *
 *   scales     host [n_scales], each in [1, 256]; n_scales in [1, 16]
 *   n_heads    >= 1;  head_dim must be 64 (else UNSUPPORTED)
 *   sm_scale   softmax scale; <= 0 selects 1/sqrt(head_dim)
 *   window     host, required
 *   share      host, may be NULL (no sharing)
 *   stream     cudaStream_t the planner kernels run on (NULL = default stream); the call
 *              synchronises that stream before it returns
 *   out_plan   receives the plan; destroy with litevar_plan_destroy
 *
 * Device work: window table (radius per step and key scale), per-axis bounds
 * [lo, hi] of every query row/column in every key scale, classification of every
 * (query tile, key tile) pair as dead / partial / full, and compaction into a per-step
 * CSR list in canonical order (query tile ascending, then key tile ascending), plus a
 * 128x128-bit element mask for every partial pair.
 * Errors: INVALID_ARG, UNSUPPORTED, EMPTY_ROW, ARCH, OOM, CUDA.
 */
litevar_status_t litevar_attn_plan(const int32_t* scales, int32_t n_scales, int32_t n_heads,
                                   int32_t head_dim, float sm_scale, const litevar_window_t* window,
                                   const litevar_cfg_share_t* share, void* stream,
                                   litevar_plan_t** out_plan);

/*
 * Step-k attention (paper Section 2 for the mask, Section 3 for sharing):
 *   out[b,h,q,:] = sum_{t live} softmax_t(sm_scale * Q[b,h,q,:] . K[b,h,t,:]) V[b,h,t,:]
 * for b in [0, 2B), h in [0, H), q in [0, n_k), t in [0, L_k); scores and sums in fp32,
 * probabilities rounded to bf16 for the PV product, output rounded to bf16.
 *
 *   step_k       1-based step
 *   batch_pairs  B; tensors hold 2B batch rows, rows [0,B) conditional, [B,2B) unconditional
 *   Q, out       device bf16 [2B, H, n_k, 64] with the given strides
 *   Kcache,Vcache device bf16 [2B, H, >= L_k, 64]; only rows [0, L_k) are read
 *   strides      in elements; each a multiple of 8; base pointers 16-byte aligned
 *   stream       cudaStream_t; the call is asynchronous, allocates nothing, synchronises nothing
 *
 * At a shared step the kernel runs for rows [0,B) only, never reads rows [B,2B) of Q/K/V,
 * and stores every output tile to rows b and b+B.  Every element of out[0..2B)[h][0..n_k)
 * is written.  Errors: INVALID_ARG (before any launch), CUDA.
 */
litevar_status_t litevar_attn_forward(const litevar_plan_t* plan, int32_t step_k, int32_t batch_pairs,
                                      const void* Q, const litevar_strides_t* sq,
                                      const void* Kcache, const litevar_strides_t* sk,
                                      const void* Vcache, const litevar_strides_t* sv,
                                      void* out, const litevar_strides_t* so, void* stream);

/*
 * Step-k attention on an 8-bit K/V cache (paper Section 4: Q, K and V in attention quantised to 8 bits, the
 * "QKV8" rows of its tables).  The cache holds, per row of a head, 64 int8 codes, a scale s and a zero point z
 * as litevar_quantize_rows produces them; a row enters the attention as code * s + z rounded to bf16.  The kernel
 * evaluates it as fma(code + 32896, s, z - 32896 s): the second operand is rounded once per row, which moves a
 * widened value by at most 2^-9 of a quantisation step s before the bf16 rounding (litevar_quantize_rows' own
 * dequantised rows round product and sum separately, so a few operands differ from them by one bf16 unit and the
 * result agrees with litevar_attn_forward on the dequantised cache closely, not bit for bit).  The cache takes 72
 * bytes per row instead of 128 and that is what the kernel reads from HBM.  Q is bf16 (quantise-dequantise it
 * with litevar_quantize_rows or litevar_quantize_qkv if the step's queries are to be 8-bit too).
 *
 *   plan, step_k, batch_pairs, Q, sq, out, so, stream   as for litevar_attn_forward
 *   Kcodes, Vcodes   device int8 [2B, H, >= L_k, 64]; strides `scodes` in bytes (= elements), each a multiple of 16,
 *                    token stride >= 64, base pointers 16-byte aligned
 *   Kscale, Kzero, Vscale, Vzero   device fp32 [2B, H, >= L_k]; strides `srow` in elements, token stride must be 1
 * Small steps run the small-step kernel, which widens the prefix while it stages it; the others run the
 * two-threads-per-row tcgen05 kernel: tensor-map copies bring the codes of a tile into the stage, three warps widen
 * them in place.  The plan must use raster tiles at this step (LITEVAR_TILING_RASTER, or AUTO at grid sides below
 * 48): else UNSUPPORTED.
 * Asynchronous, allocates nothing.  Errors: INVALID_ARG (before any launch), UNSUPPORTED, CUDA.
 */
litevar_status_t litevar_attn_forward_kv8(const litevar_plan_t* plan, int32_t step_k, int32_t batch_pairs,
                                          const void* Q, const litevar_strides_t* sq, const int8_t* Kcodes,
                                          const float* Kscale, const float* Kzero, const int8_t* Vcodes,
                                          const float* Vscale, const float* Vzero, const litevar_strides_t* scodes,
                                          const litevar_strides_t* srow, void* out, const litevar_strides_t* so,
                                          void* stream);

/*
 * Step-k attention without a plan object and without any allocation.  The paper has no counterpart:
 * this is a deployment convenience of this library.
 *
 * litevar_attn_plan keeps its tile lists in memory it gets from cudaMalloc.  A caller that may not
 * allocate (it runs inside a fixed device-memory budget, it is a plug-in that must stay away from its
 * host's allocator, or it is reached at a point where allocation is forbidden) uses this call instead:
 * it builds the tile plan of step_k on the device inside a fixed 4.2 MB array that is part of the
 * library image, then runs the same tensor-core forward kernel on it.  It calls no cudaMalloc, no
 * cudaFree and no allocating library routine; it launches three kernels on `stream` and returns
 * without synchronising.
 *
 *   scales .. sm_scale, window   as for litevar_attn_plan (window->n_sets must be 1; a radius table,
 *                                if given, is read at row step_k-1 only; head_to_set is ignored)
 *   share_cfg                    non-zero: CFG sharing at this step (rows [0,B) computed, stored twice)
 *   step_k .. stream             as for litevar_attn_forward
 *
 * Limits and rules.
 *   - The step must have at most 2048 candidate tile pairs, ceil(n_k/128) * ceil(L_k/128)
 *     (every step of the 256px and 512px schedules fits; the 2K step does not): otherwise
 *     LITEVAR_ERR_UNSUPPORTED is returned and nothing is launched.
 *   - Every GPU that loads the library holds the array until the process exits.  All calls on a device
 *     share it and it keeps the last call's contents: calls that may overlap on the GPU (different
 *     streams, or concurrent host threads) race; keep them on one stream or order them yourself.
 *     Each call rewrites every entry it later reads and clears its status word, so nothing depends on
 *     what an earlier call left behind.
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress) with
 *     that device current; make that first call outside any stream capture.
 *   - There is no empty-row check: with a caller table that leaves a query without a live key the
 *     row's output is undefined.  A bounded device-side wait that expires is not reported.
 * Errors: INVALID_ARG, UNSUPPORTED, ARCH, CUDA.  (A tensor-map encoding failure, INVALID_ARG, is found after the two
 * planner kernels have been launched; they write only the library's own array.)
 */
litevar_status_t litevar_attn_forward_static(const int32_t* scales, int32_t n_scales, int32_t n_heads,
                                             int32_t head_dim, float sm_scale, const litevar_window_t* window,
                                             int32_t share_cfg, int32_t step_k, int32_t batch_pairs,
                                             const void* Q, const litevar_strides_t* sq,
                                             const void* Kcache, const litevar_strides_t* sk,
                                             const void* Vcache, const litevar_strides_t* sv,
                                             void* out, const litevar_strides_t* so, void* stream);

/*
 * Window calibration of one step (paper Section 2, "detailed process of the MDWA pattern design", steps
 * (1)-(3)): given saved post-softmax attention maps of step k, find for every part j after the global ones
 * the smallest window radius w whose ratio R_w (sum of the map inside the window / sum of the whole part,
 * taken over all given maps and query rows) reaches the threshold R_0.  Square windows only.
 *
 *   maps     device float32 [n_maps][n_k][L_k], contiguous, non-negative (rows need not sum to 1)
 *   r0       threshold R_0 in (0, 1]; the decision is window mass >= r0 * part mass in fp64
 *   radius   host out [n_scales]: -1 for parts j <= n_global_scales and for j > step_k, else the radius;
 *            a row of this kind is what litevar_window_t.radius takes
 *   ratio    host out [n_scales][256] or NULL: R_w for w = 0 .. s_j - 1 (1 elsewhere)
 *   stream   the kernel runs there; the call synchronises the stream and allocates 32 KB of scratch
 * One pass over the maps (the kernel is bound by reading them once).
 * Errors: INVALID_ARG, OOM, CUDA.
 */
litevar_status_t litevar_calibrate_windows(const int32_t* scales, int32_t n_scales, int32_t step_k,
                                           int32_t n_global_scales, const float* maps, int64_t n_maps, double r0,
                                           int32_t* radius, double* ratio, void* stream);

/* Counts for step k and window set `set`: live map entries, live / full / partial tile pairs. */
litevar_status_t litevar_plan_stats(const litevar_plan_t* plan, int32_t step_k, int32_t set,
                                    int64_t* live_entries, int64_t* live_tiles, int64_t* full_tiles,
                                    int64_t* partial_tiles);

/* Sizes of the step-k tile plan of one window set. */
litevar_status_t litevar_plan_tile_counts(const litevar_plan_t* plan, int32_t step_k, int32_t set,
                                          int32_t* n_q_tiles, int32_t* n_key_tiles, int32_t* n_pairs);

/*
 * Copy the step-k tile plan to host arrays sized from litevar_plan_tile_counts (any may be NULL):
 *   q_tile_geom   [n_q_tiles][5]   {first token, columns, row stride, valid rows, valid columns}: slot m
 *                                  (0 <= m < 128) sits at row m / columns, column m % columns of the tile; it
 *                                  holds token first + row * row_stride + column when row < valid rows and
 *                                  column < valid columns, and is padding otherwise (raster tiles: one row of
 *                                  128 columns; patch tiles: 8 rows of 16 columns, row stride = grid side)
 *   key_tile_geom [n_key_tiles][5] same, tokens index the K/V cache
 *   row_ptr       [n_q_tiles + 1]  CSR offsets into the pair arrays
 *   pair_key_tile [n_pairs]        key tile of each live pair, ascending inside a query tile
 *   pair_is_full  [n_pairs]        1 = every slot pair live (no element mask), 0 = partial
 */
litevar_status_t litevar_plan_export_tiles(const litevar_plan_t* plan, int32_t step_k, int32_t set,
                                           int32_t* q_tile_geom, int32_t* key_tile_geom,
                                           int32_t* row_ptr, int32_t* pair_key_tile,
                                           uint8_t* pair_is_full);

/* Copy the window radii of step k (host out [n_scales], -1 = global, entries j > k are -1) and the
 * per-axis bounds the device computed (host out [step_k][s_k][2] int32: lo, hi of query row or
 * column x in key scale j; SQUARE windows only; either pointer may be NULL). */
litevar_status_t litevar_plan_export_bounds(const litevar_plan_t* plan, int32_t step_k, int32_t set,
                                            int32_t* radius, int32_t* bounds);

/* Expand the tile list and element masks of step k into a dense bit mask on the device:
 * dev_bits is n_k rows of ceil(L_k / 32) uint32 words, bit (t & 31) of word t >> 5 = live(q, t).
 * Runs on `stream`, asynchronous.  The mask blocks read here are the ones the attention kernel reads. */
litevar_status_t litevar_plan_materialize_mask(const litevar_plan_t* plan, int32_t step_k, int32_t set,
                                               void* dev_bits, void* stream);

/* Synchronises the device and reports LITEVAR_ERR_DEVICE_TIMEOUT if any forward kernel launched
 * with this plan gave up on a bounded wait since the last poll (the flag is then cleared). */
litevar_status_t litevar_plan_poll_device_status(const litevar_plan_t* plan);

/* Testing and measurement hook: force one forward kernel for every step (LITEVAR_KERNEL_SIMT, _TCGEN05,
 * _TCGEN05_WS) or return to LITEVAR_KERNEL_AUTO, which is what a plan starts with and all a product caller needs.
 * Changes the plan: not to be called while forwards of this plan may be running or being issued. */
litevar_status_t litevar_plan_set_kernel(litevar_plan_t* plan, int32_t kernel);

/* Which kernel litevar_attn_forward launches for step_k with batch_pairs under the current selection:
 * *kernel receives LITEVAR_KERNEL_SIMT, _TCGEN05, _TCGEN05_WS or _SMALL.  Host only; the paper has no counterpart (it gives no kernel design). */
litevar_status_t litevar_plan_step_kernel(const litevar_plan_t* plan, int32_t step_k, int32_t batch_pairs,
                                          int32_t* kernel);

/*
 * 8-bit Q/K/V (paper Section 4, dynamic quantisation): quantise every token row of a head (head_dim values) of
 * a bf16 tensor x[batch][n_heads][n_tokens][head_dim] (element strides sx, head_dim contiguous) to `bits`-bit
 * integers with a scale and a zero point taken from the row's maximum and minimum:
 *     z = (max + min) / 2,  s = (max - min) / (2^bits - 1),
 *     code = clamp(round((x - z) / s), -2^(bits-1), 2^(bits-1) - 1)   (round to nearest even; s = 0: code 0),
 *     all in fp32, one correctly rounded IEEE operation at a time (the quotient is an IEEE division).  Outputs, each optional (NULL = not wanted), all device memory:
 *   x_dq   bf16, strides sdq: the dequantised rows code * s + z rounded to bf16 - what the attention then reads;
 *          may be x itself (in place)
 *   codes  int8 [batch][n_heads][n_tokens][head_dim], dense, 8-byte aligned
 *   scale, zero  fp32 [batch][n_heads][n_tokens], dense
 * Granularity (per token row) and the step s are readings of the paper, which prints s = max(abs(x)) beside
 * clamp bounds that do not match it.  Asynchronous on `stream`, allocates nothing, graph-capturable.
 * Errors: NULL x, bad strides or alignment, batch / n_heads / n_tokens < 1, bits outside 2..8 -> INVALID_ARG;
 * head_dim != 64 -> UNSUPPORTED.  Pointers are borrowed.
 */
litevar_status_t litevar_quantize_rows(const void* x, const litevar_strides_t* sx, int32_t batch, int32_t n_heads,
                                       int32_t n_tokens, int32_t head_dim, int32_t bits, void* x_dq,
                                       const litevar_strides_t* sdq, int8_t* codes, float* scale, float* zero,
                                       void* stream);

/*
 * The same quantiser for the three tensors of one attention call, in place, in one launch: the step's Q
 * (n_q_tokens rows per head) and the K and V rows appended to the cache at this step (n_kv_tokens rows per head
 * each; pass pointers to the first appended row).  Every row is replaced by its dequantised value, which is what
 * litevar_attn_forward then reads (paper Section 4: Q, K and V in attention quantised to 8 bits).  Launched
 * with programmatic stream serialisation, so that its launch overlaps the previous kernel of the stream; it
 * waits for that kernel before it reads.  Errors as litevar_quantize_rows.
 */
litevar_status_t litevar_quantize_qkv(void* q, const litevar_strides_t* sq, int32_t n_q_tokens, void* k,
                                      const litevar_strides_t* sk, void* v, const litevar_strides_t* sv,
                                      int32_t n_kv_tokens, int32_t batch, int32_t n_heads, int32_t head_dim,
                                      int32_t bits, void* stream);

/* Frees the plan and its device buffers.  NULL is allowed. */
void litevar_plan_destroy(litevar_plan_t* plan);

/* Static string for a status code. */
const char* litevar_status_string(litevar_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* LITEVAR_H_ */
