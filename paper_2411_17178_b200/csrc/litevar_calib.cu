// Window calibration of one step (paper Section 2, steps (1)-(3)): from saved post-softmax attention maps,
// for every part of the step-k map find the smallest window radius w whose share R_w of the part's
// attention mass reaches the threshold R_0.
//
// R_w for all w at once: every map entry (q, t) of part j lies at Chebyshev distance
// d = max(|r' - ctr_j(r)|, |c' - ctr_j(c)|) from the key cell under the query; the window of radius w holds
// exactly the entries with d <= w.  One pass over the maps accumulates the mass per (part, distance); a
// running sum over d then gives the window mass for every w.  The pass is bound by reading the maps once.
//
// A warp owns batches of consecutive (map, query) rows and walks them once per part, so that it needs
// histogram bins for one part at a time: bins[distance][lane] in shared memory (fp32), private to the lane,
// updated with plain loads and stores.  After at most 256 rows the bins are summed over the lanes in fp64 and
// added to the global histogram with one fp64 add per non-empty bin.
//   Parts of up to 256 keys: a lane reads flat key positions t = 32 * chunk + lane, so every lane of a load is
// used whatever the grid width, and one round takes the same chunk of eight query rows (eight independent
// loads in flight however small the part).
//   Wider parts: lanes sweep the columns of a key row.  In a key row at row distance dr the entries whose
// column distance is smaller fall into bin dr and add up in a register before one shared-memory update per
// key row; the others belong to the bin of their own column distance, which is fixed per lane, so they add up
// in registers over all key rows of the query.
#include <cuda_runtime.h>

#include <cstring>
#include <vector>

#include "litevar_internal.h"

namespace litevar {

namespace {

constexpr int kCalibWarps = 4;
constexpr int kMaxDist = kMaxScale;   // distances 0 .. s_j - 1
constexpr int kCalibFlushRows = 256;  // rows a lane's fp32 bins take in before they are flushed
constexpr int kCalibMaxRows = 1 << 30;  // (map, query) rows of one launch

// Wide part (more than 256 keys) of one query row: NC 32-column chunks per key row, 16 loads in flight per round.
template <int NC>
__device__ __forceinline__ void calib_wide_row(float* bins, int lane, const float* __restrict__ part, int s_j, int cr,
                                               int cc) {
  constexpr int KR = 16 / NC;
  int dc[NC];
  float outer[NC];
  bool cv[NC];
#pragma unroll
  for (int u = 0; u < NC; ++u) {
    const int kc = lane + 32 * u;
    cv[u] = kc < s_j;
    dc[u] = abs(kc - cc);
    outer[u] = 0.f;
  }
  for (int kr0 = 0; kr0 < s_j; kr0 += KR) {
    float a[KR][NC];
#pragma unroll
    for (int v = 0; v < KR; ++v)
#pragma unroll
      for (int u = 0; u < NC; ++u)
        a[v][u] = (cv[u] && kr0 + v < s_j) ? __ldg(part + (kr0 + v) * s_j + lane + 32 * u) : 0.f;
#pragma unroll
    for (int v = 0; v < KR; ++v) {
      const int kr = kr0 + v;
      if (kr < s_j) {
        const int dr = abs(kr - cr);
        float inner = 0.f;
#pragma unroll
        for (int u = 0; u < NC; ++u) {
          if (dc[u] < dr) inner += a[v][u]; else outer[u] += a[v][u];
        }
        bins[(dr << 5) + lane] += inner;
      }
    }
  }
#pragma unroll
  for (int u = 0; u < NC; ++u)
    if (cv[u]) bins[(dc[u] << 5) + lane] += outer[u];
}

__global__ void __launch_bounds__(kCalibWarps * 32, 32 / kCalibWarps)
calib_hist_kernel(Schedule sc, int k0, int first_part, int s_max, const float* __restrict__ maps, int n_rows_total,
                  int q_first /* query index of row 0 */, int rows_per_batch,
                  double* __restrict__ hist /* [kMaxScales][kMaxDist] */) {
  extern __shared__ float sh[];  // [kCalibWarps][s_max][32]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* bins = sh + (size_t)warp * s_max * 32;
  const int s_k = sc.scale[k0];
  const int n_k = s_k * s_k;
  const int L_k = sc.off[k0 + 1];
  const int n_batches = (n_rows_total + rows_per_batch - 1) / rows_per_batch;
  const int warp_global = blockIdx.x * kCalibWarps + warp;
  const int n_warps = gridDim.x * kCalibWarps;
  const int flush_every = max(1, kCalibFlushRows / rows_per_batch);

  for (int j = first_part; j <= k0; ++j) {
    const int s_j = sc.scale[j];
    const int n_j = s_j * s_j;
    const int n_chunks = (n_j + 31) >> 5;
    const int step_r = 32 / s_j, step_c = 32 - step_r * s_j;  // a lane's flat key cell moves by this per chunk
    const int r_t0 = lane / s_j, c_t0 = lane - r_t0 * s_j;
    const int off_j = sc.off[j];
    double* hist_j = hist + (size_t)j * kMaxDist;
    for (int d = 0; d < s_j; ++d) bins[(d << 5) + lane] = 0.f;
    int pending = 0;
    for (int batch = warp_global; batch < n_batches; batch += n_warps) {
      const int row0 = batch * rows_per_batch;
      const int nb = min(rows_per_batch, n_rows_total - row0);
      // lane i holds the co-located key cell of row i of the batch
      int pk;
      {
        const unsigned q = ((unsigned)(q_first + row0 % n_k) + (unsigned)lane) % (unsigned)n_k;
        const int r = (int)q / s_k, c = (int)q - r * s_k;
        pk = (((2 * r + 1) * s_j) / (2 * s_k)) | ((((2 * c + 1) * s_j) / (2 * s_k)) << 16);
      }
      const float* src = maps + (size_t)row0 * L_k + off_j;
      if (n_chunks <= 8) {
        for (int i0 = 0; i0 < nb; i0 += 8) {
          int cr[8], cc[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int p = __shfl_sync(0xffffffffu, pk, (i0 + u) & 31);
            cr[u] = p & 0xffff;
            cc[u] = p >> 16;
          }
          const int ng = nb - i0;
          const float* grp = src + (size_t)i0 * L_k + lane;
          int r_t = r_t0, c_t = c_t0;
          for (int ch = 0; ch < n_chunks; ++ch) {
            const bool tv = (ch << 5) + lane < n_j;
            float a[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) a[u] = (tv && u < ng) ? __ldg(grp + (size_t)u * L_k + (ch << 5)) : 0.f;
            if (tv) {
              // rows past the end of the batch carry zeros into a valid bin
#pragma unroll
              for (int u = 0; u < 8; ++u)
                bins[(max(abs(r_t - cr[u]), abs(c_t - cc[u])) << 5) + lane] += a[u];
            }
            r_t += step_r;
            c_t += step_c;
            if (c_t >= s_j) {
              c_t -= s_j;
              ++r_t;
            }
          }
        }
      } else {
        const int nc = (s_j + 31) >> 5;
        for (int i = 0; i < nb; ++i) {
          const int p = __shfl_sync(0xffffffffu, pk, i);
          const int cr = p & 0xffff, cc = p >> 16;
          const float* part = src + (size_t)i * L_k;
          switch (nc) {
            case 1: calib_wide_row<1>(bins, lane, part, s_j, cr, cc); break;
            case 2: calib_wide_row<2>(bins, lane, part, s_j, cr, cc); break;
            case 3: calib_wide_row<3>(bins, lane, part, s_j, cr, cc); break;
            case 4: calib_wide_row<4>(bins, lane, part, s_j, cr, cc); break;
            default: calib_wide_row<8>(bins, lane, part, s_j, cr, cc); break;
          }
        }
      }
      if (++pending == flush_every || batch + n_warps >= n_batches) {
        pending = 0;
        __syncwarp();
        // lane l sums bin d = d0 + l over the 32 lane columns, rotated so that the lanes hit distinct banks
        for (int d0 = 0; d0 < s_j; d0 += 32) {
          const int d = d0 + lane;
          if (d < s_j) {
            double sum = 0.0;
#pragma unroll 8
            for (int i = 0; i < 32; ++i) sum += (double)bins[(d << 5) + ((i + lane) & 31)];
            if (sum != 0.0) atomicAdd(&hist_j[d], sum);
          }
        }
        __syncwarp();
        for (int d = 0; d < s_j; ++d) bins[(d << 5) + lane] = 0.f;
      }
    }
    __syncwarp();
  }
}

}  // namespace

}  // namespace litevar

using namespace litevar;

extern "C" litevar_status_t litevar_calibrate_windows(const int32_t* scales, int32_t n_scales, int32_t step_k,
                                                      int32_t n_global_scales, const float* maps, int64_t n_maps,
                                                      double r0, int32_t* radius, double* ratio, void* stream_) {
  if (!scales || !maps || !radius) return LITEVAR_ERR_INVALID_ARG;
  if (n_scales < 1 || n_scales > kMaxScales || step_k < 1 || step_k > n_scales || n_maps < 1 ||
      n_global_scales < 0 || !(r0 > 0.0) || r0 > 1.0)
    return LITEVAR_ERR_INVALID_ARG;
  for (int i = 0; i < n_scales; ++i)
    if (scales[i] < 1 || scales[i] > kMaxScale) return LITEVAR_ERR_INVALID_ARG;
  if ((uintptr_t)maps & 3) return LITEVAR_ERR_INVALID_ARG;
  Schedule sc;
  memset(&sc, 0, sizeof(sc));
  sc.n_scales = n_scales;
  for (int i = 0; i < n_scales; ++i) {
    sc.scale[i] = scales[i];
    sc.off[i + 1] = sc.off[i] + scales[i] * scales[i];
  }
  const int k0 = step_k - 1;
  const int first_part = n_global_scales < step_k ? n_global_scales : step_k;
  for (int j = 0; j < n_scales; ++j) radius[j] = -1;
  if (ratio)
    for (int i = 0; i < n_scales * kMaxDist; ++i) ratio[i] = 1.0;
  if (first_part > k0) return LITEVAR_OK;  // every part of this step is global

  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  double* d_hist = nullptr;
  const size_t hist_bytes = sizeof(double) * kMaxScales * kMaxDist;
  if (cudaMallocAsync(&d_hist, hist_bytes, stream) != cudaSuccess) {
    (void)cudaGetLastError();
    return LITEVAR_ERR_OOM;
  }
  litevar_status_t st = LITEVAR_OK;
  std::vector<double> hist((size_t)kMaxScales * kMaxDist);
  const int n_k = scales[k0] * scales[k0];
  const long long rows = (long long)n_maps * n_k;
  const long long L_k = sc.off[k0 + 1];
  int dev = 0, n_sm = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) (void)cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
  int s_max = 1;
  for (int j = first_part; j <= k0; ++j) s_max = scales[j] > s_max ? scales[j] : s_max;
  const size_t smem = sizeof(float) * 32 * (size_t)s_max * kCalibWarps;
  // resident warps: up to 32 per SM, fewer where the bins of the widest part need the shared memory
  int blocks_per_sm = (int)((200u << 10) / (smem + 1024));
  if (blocks_per_sm > 32 / kCalibWarps) blocks_per_sm = 32 / kCalibWarps;
  if (blocks_per_sm < 1) blocks_per_sm = 1;
  const long long n_warps = (long long)n_sm * blocks_per_sm * kCalibWarps;
  if (cudaMemsetAsync(d_hist, 0, hist_bytes, stream) != cudaSuccess ||
      cudaFuncSetAttribute(calib_hist_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    st = LITEVAR_ERR_CUDA;
  for (long long first = 0; first < rows && st == LITEVAR_OK; first += kCalibMaxRows) {
    const int n_rows = (int)(rows - first < kCalibMaxRows ? rows - first : kCalibMaxRows);
    // rows per batch: the choice whose batch waves over the resident warps finish first, counting a batch
    // as the mean of its rows (wide parts) and its rows rounded up to groups of eight (small parts)
    int rows_per_batch = 1;
    long long best = 0;
    for (int rpb = 32; rpb >= 1; --rpb) {
      const long long batches = (n_rows + rpb - 1) / rpb;
      const long long span = (batches + n_warps - 1) / n_warps * (rpb + (rpb + 7) / 8 * 8);
      if (best == 0 || span < best) {
        best = span;
        rows_per_batch = rpb;
      }
    }
    const long long n_batches = ((long long)n_rows + rows_per_batch - 1) / rows_per_batch;
    long long blocks = (n_batches + kCalibWarps - 1) / kCalibWarps;
    if (blocks > (long long)n_sm * blocks_per_sm) blocks = (long long)n_sm * blocks_per_sm;
    calib_hist_kernel<<<(unsigned)blocks, kCalibWarps * 32, smem, stream>>>(
        sc, k0, first_part, s_max, maps + first * L_k, n_rows, (int)(first % n_k), rows_per_batch, d_hist);
    if (cudaGetLastError() != cudaSuccess) st = LITEVAR_ERR_CUDA;
  }
  if (st == LITEVAR_OK && (cudaMemcpyAsync(hist.data(), d_hist, hist_bytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
                           cudaStreamSynchronize(stream) != cudaSuccess))
    st = LITEVAR_ERR_CUDA;
  (void)cudaFreeAsync(d_hist, stream);
  if (st != LITEVAR_OK) {
    (void)cudaGetLastError();
    return st;
  }
  // running sums over the distance: window mass for every radius; smallest radius with mass >= R_0 * total
  for (int j = first_part; j <= k0; ++j) {
    const double* h = hist.data() + (size_t)j * kMaxDist;
    double total = 0.0;
    for (int d = 0; d < scales[j]; ++d) total += h[d];
    double cum = 0.0;
    int w = scales[j] - 1;
    bool found = false;
    for (int d = 0; d < scales[j]; ++d) {
      cum += h[d];
      if (ratio) ratio[(size_t)j * kMaxDist + d] = total > 0.0 ? cum / total : 1.0;
      if (!found && cum >= r0 * total) {
        w = d;
        found = true;
      }
    }
    radius[j] = w;
  }
  return LITEVAR_OK;
}
