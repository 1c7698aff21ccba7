// Window calibration of one step (paper Section 2, steps (1)-(3)): from saved post-softmax attention maps,
// for every part of the step-k map find the smallest window radius w whose share R_w of the part's
// attention mass reaches the threshold R_0.
//
// R_w for all w at once: every map entry (q, t) of part j lies at Chebyshev distance
// d = max(|r' - ctr_j(r)|, |c' - ctr_j(c)|) from the key cell under the query; the window of radius w holds
// exactly the entries with d <= w.  One pass over the maps accumulates the mass per (part, distance); a
// running sum over d then gives the window mass for every w.  The pass is bound by reading the maps once.
//
// One warp per (map, query row); lanes sweep a key row of the part.  In a key row at row distance dr all
// entries whose column distance is <= dr fall into bin dr (one warp reduction, one shared-memory add), the
// others into the bin of their own column distance (at most two lanes per bin).  Block histograms in shared
// memory (fp64) are flushed with one global fp64 add per non-empty bin.
#include <cuda_runtime.h>

#include <cstring>
#include <vector>

#include "litevar_internal.h"

namespace litevar {

namespace {

constexpr int kCalibWarps = 8;
constexpr int kMaxDist = kMaxScale;  // distances 0 .. s_j - 1

__global__ void __launch_bounds__(kCalibWarps * 32)
calib_hist_kernel(Schedule sc, int k0, int first_part, const float* __restrict__ maps, long long n_rows_total,
                  double* __restrict__ hist /* [kMaxScales][kMaxDist] */) {
  extern __shared__ double sh[];  // [(k0 + 1 - first_part)][s_max] bins of this block
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int s_k = sc.scale[k0];
  const int n_k = s_k * s_k;
  const int L_k = sc.off[k0 + 1];
  const int n_parts = k0 + 1 - first_part;
  for (int i = threadIdx.x; i < n_parts * kMaxDist; i += blockDim.x) sh[i] = 0.0;
  __syncthreads();
  for (long long row = (long long)blockIdx.x * kCalibWarps + warp; row < n_rows_total;
       row += (long long)gridDim.x * kCalibWarps) {
    const int q = (int)(row % n_k);
    const int r = q / s_k, c = q - r * s_k;
    const float* src = maps + row * L_k;
    for (int j = first_part; j <= k0; ++j) {
      const int s_j = sc.scale[j];
      const int cr = ((2 * r + 1) * s_j) / (2 * s_k), cc = ((2 * c + 1) * s_j) / (2 * s_k);
      double* bins = sh + (size_t)(j - first_part) * kMaxDist;
      const float* part = src + sc.off[j];
      for (int kr = 0; kr < s_j; ++kr) {
        const int dr = kr > cr ? kr - cr : cr - kr;
        float inner = 0.f;  // entries of this key row that belong to bin dr
        for (int kc = lane; kc < s_j; kc += 32) {
          const float a = __ldg(part + kr * s_j + kc);
          const int dc = kc > cc ? kc - cc : cc - kc;
          if (dc <= dr)
            inner += a;
          else if (a != 0.f)
            atomicAdd(&bins[dc], (double)a);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) inner += __shfl_xor_sync(0xffffffffu, inner, o);
        if (lane == 0 && inner != 0.f) atomicAdd(&bins[dr], (double)inner);
      }
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < n_parts * kMaxDist; i += blockDim.x) {
    const double v = sh[i];
    if (v != 0.0) atomicAdd(&hist[(size_t)(first_part + i / kMaxDist) * kMaxDist + i % kMaxDist], v);
  }
}

}  // namespace

}  // namespace litevar

using namespace litevar;

extern "C" litevar_status_t litevar_calibrate_windows(const int32_t* scales, int32_t n_scales, int32_t step_k,
                                                      int32_t n_global_scales, const float* maps, int64_t n_maps,
                                                      float r0, int32_t* radius, double* ratio, void* stream_) {
  if (!scales || !maps || !radius) return LITEVAR_ERR_INVALID_ARG;
  if (n_scales < 1 || n_scales > kMaxScales || step_k < 1 || step_k > n_scales || n_maps < 1 ||
      n_global_scales < 0 || !(r0 > 0.f) || r0 > 1.f)
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
  if (cudaMalloc(&d_hist, hist_bytes) != cudaSuccess) {
    (void)cudaGetLastError();
    return LITEVAR_ERR_OOM;
  }
  litevar_status_t st = LITEVAR_OK;
  std::vector<double> hist((size_t)kMaxScales * kMaxDist);
  const long long rows = (long long)n_maps * scales[k0] * scales[k0];
  int dev = 0, n_sm = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) (void)cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
  long long blocks = (rows + kCalibWarps - 1) / kCalibWarps;
  if (blocks > 8LL * n_sm) blocks = 8LL * n_sm;  // grid-stride: a few resident blocks per SM keep the flush cheap
  const size_t smem = sizeof(double) * (size_t)(k0 + 1 - first_part) * kMaxDist;
  if (cudaMemsetAsync(d_hist, 0, hist_bytes, stream) != cudaSuccess ||
      cudaFuncSetAttribute(calib_hist_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
    st = LITEVAR_ERR_CUDA;
  } else {
    calib_hist_kernel<<<(unsigned)blocks, kCalibWarps * 32, smem, stream>>>(sc, k0, first_part, maps, rows, d_hist);
    if (cudaGetLastError() != cudaSuccess ||
        cudaMemcpyAsync(hist.data(), d_hist, hist_bytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess)
      st = LITEVAR_ERR_CUDA;
  }
  cudaFree(d_hist);
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
      if (!found && cum >= (double)r0 * total) {
        w = d;
        found = true;
      }
    }
    radius[j] = w;
  }
  return LITEVAR_OK;
}
