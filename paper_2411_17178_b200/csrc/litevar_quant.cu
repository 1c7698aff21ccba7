// Dynamic min-max quantisation of Q, K or V rows to B-bit integers (paper Section 4, "QKV8"): for every token
// row of a head (64 values) z = (max + min) / 2, s = (max - min) / (2^B - 1),
// code = clamp(round((x - z) / s), -2^(B-1), 2^(B-1) - 1), and the attention runs on code * s + z.  The code is
// the one the correctly rounded fp32 quotient (x - z) / s gives: the quotient is first estimated as
// (x - z) * (1 / s), which is within two units in the last place of it; only an estimate that close to a
// rounding tie (a half-integer) can round to another integer than the quotient does, and those few elements
// take the IEEE division.
//
// In a generation the rows of a step are quantised once, when they are appended to the K/V cache (and Q as it
// is produced); the attention kernels then read the dequantised bf16 rows unchanged.  The pass is bound by
// reading and writing each row once: eight threads share a row (16 bytes each) and take up to four rows at a
// time (four loads in flight), the row's maximum and minimum come from three shuffles, every thread codes and
// rebuilds its own eight values.  It may run in place.
//
// The integer decision is taken in fp32 with one IEEE operation at a time (no contraction into fused
// multiply-adds), so that it can be reproduced exactly.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "litevar_internal.h"

namespace litevar {

namespace {

constexpr int kQuantThreads = 256;

// One tensor of a launch: rows [first_row, first_row + batch * n_heads * n_tokens) of the launch's row space.
struct QuantTensor {
  const uint16_t* x;
  uint16_t* dq;  // nullptr: no dequantised output
  int64_t x_sb, x_sh, x_st, d_sb, d_sh, d_st;
  int32_t n_tokens;
  long long first_row;
};
struct QuantArgs {
  QuantTensor t[3];
  int32_t n_tensors, n_heads;
  long long n_rows;
  float levels, lo, hi;
  int8_t* codes;  // outputs of the first tensor only
  float* scale;
  float* zero;
};

// kQuantRowsPerGroup rows per 8-thread group: that many 16-byte loads in flight per thread.  Four for large
// tensors (bandwidth), one for the few rows of a single step (more threads, shorter latency chain).
template <int kQuantRowsPerGroup>
__global__ void __launch_bounds__(kQuantThreads, 4) quant_rows_kernel(QuantArgs a) {
  // the rows were written by earlier work of the stream; a launch with programmatic serialisation starts early
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int part = threadIdx.x & 7;  // 16-byte column of the row
  // rows [R * group, R * group + R) per eight threads, no loop: the grid covers the rows (fewer than 2^31,
  // checked on the host).  Slots past the last row redo the last row and store nothing, so that every lane
  // joins the shuffles.
  const unsigned group = blockIdx.x * (unsigned)(kQuantThreads / 8) + (threadIdx.x >> 3);
  bool valid[kQuantRowsPerGroup];
  unsigned row[kQuantRowsPerGroup];
  int ti[kQuantRowsPerGroup];
  int64_t x_off[kQuantRowsPerGroup], d_off[kQuantRowsPerGroup];
  uint4 raw[kQuantRowsPerGroup];
#pragma unroll
  for (int g = 0; g < kQuantRowsPerGroup; ++g) {
    const unsigned slot = group * kQuantRowsPerGroup + g;
    valid[g] = slot < (unsigned)a.n_rows;
    row[g] = valid[g] ? slot : (unsigned)a.n_rows - 1u;
    ti[g] = 0;
    if (a.n_tensors > 1 && row[g] >= (unsigned)a.t[1].first_row) ti[g] = 1;
    if (a.n_tensors > 2 && row[g] >= (unsigned)a.t[2].first_row) ti[g] = 2;
    const QuantTensor& tn = a.t[ti[g]];
    const unsigned local = row[g] - (unsigned)tn.first_row;
    const unsigned bh = local / (unsigned)tn.n_tokens;
    const int t = (int)(local - bh * (unsigned)tn.n_tokens);
    const unsigned b = bh / (unsigned)a.n_heads;
    const int h = (int)(bh - b * (unsigned)a.n_heads);
    x_off[g] = b * tn.x_sb + h * tn.x_sh + (int64_t)t * tn.x_st + part * 8;
    d_off[g] = b * tn.d_sb + h * tn.d_sh + (int64_t)t * tn.d_st + part * 8;
    raw[g] = *reinterpret_cast<const uint4*>(tn.x + x_off[g]);
  }
#pragma unroll
  for (int g = 0; g < kQuantRowsPerGroup; ++g) {
    const QuantTensor& tn = a.t[ti[g]];
    const uint32_t u[4] = {raw[g].x, raw[g].y, raw[g].z, raw[g].w};
    float v[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(u[i] << 16);
      v[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
    }
    float mx = v[0], mn = v[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) {
      mx = fmaxf(mx, v[i]);
      mn = fminf(mn, v[i]);
    }
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) {  // the eight threads of a row are adjacent lanes
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
    }
    const float z = __fmul_rn(__fadd_rn(mx, mn), 0.5f);
    const float s = __fdiv_rn(__fsub_rn(mx, mn), a.levels);
    const float s1 = s > 0.f ? s : 1.f;
    const float r = __fdiv_rn(1.f, s1);  // one division per row; the elements multiply, see below
    float c[8];
    uint32_t packed[4];
    // round to nearest even without the conversion pipe: adding and subtracting 1.5 * 2^23 is exact rounding
    // to an integer for |y| < 2^22, and |y| stays near 2^(B-1) here.  The estimate y = (x - z) * (1 / s) is within
    // |y| * 2^-23 < 2^-15.9 of the true quotient and the correctly rounded quotient within 2^-17 of it, so an
    // estimate farther than 2^-14 from a half-integer rounds as the IEEE quotient does; a thread with an estimate
    // closer than that redoes its eight values with the division.  So does every thread of a row whose step is so
    // small that its reciprocal is not a normal number.
    bool divide = !(s1 > 1e-30f);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float y = __fmul_rn(__fsub_rn(v[i], z), r);
      const float n = __fsub_rn(__fadd_rn(y, 12582912.f), 12582912.f);
      divide |= fabsf(__fsub_rn(y, n)) > 0.5f - 0.00006103515625f;
      c[i] = n;
    }
    if (divide) {  // rare (one thread-row in a thousand): all eight values again, with the IEEE division
#pragma unroll
      for (int i = 0; i < 8; ++i)
        c[i] = __fsub_rn(__fadd_rn(__fdiv_rn(__fsub_rn(v[i], z), s1), 12582912.f), 12582912.f);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) c[i] = s > 0.f ? fminf(fmaxf(c[i], a.lo), a.hi) : 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 d2 = __floats2bfloat162_rn(__fadd_rn(__fmul_rn(c[2 * i], s), z),
                                                      __fadd_rn(__fmul_rn(c[2 * i + 1], s), z));
      packed[i] = *reinterpret_cast<const uint32_t*>(&d2);
    }
    if (valid[g] && tn.dq != nullptr)
      *reinterpret_cast<uint4*>(tn.dq + d_off[g]) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
    if (valid[g] && ti[g] == 0) {
      if (a.codes != nullptr) {
        uint32_t w[2];
#pragma unroll
        for (int i = 0; i < 2; ++i)
          w[i] = ((uint32_t)(int)c[4 * i] & 0xffu) | (((uint32_t)(int)c[4 * i + 1] & 0xffu) << 8) |
                 (((uint32_t)(int)c[4 * i + 2] & 0xffu) << 16) | (((uint32_t)(int)c[4 * i + 3] & 0xffu) << 24);
        *reinterpret_cast<uint2*>(a.codes + (size_t)row[g] * kHeadDim + part * 8) = make_uint2(w[0], w[1]);
      }
      if (part == 0) {
        if (a.scale != nullptr) a.scale[row[g]] = s;
        if (a.zero != nullptr) a.zero[row[g]] = z;
      }
    }
  }
}

bool quant_strides_ok(const litevar_strides_t* s) {
  return s && s->batch >= 0 && s->head >= 0 && s->token >= kHeadDim && (s->batch % 8) == 0 && (s->head % 8) == 0 &&
         (s->token % 8) == 0;
}

litevar_status_t launch_quant(QuantArgs& a, int bits, bool overlap, cudaStream_t stream) {
  a.levels = (float)((1 << bits) - 1);
  a.lo = -(float)(1 << (bits - 1));
  a.hi = (float)((1 << (bits - 1)) - 1);
  if (a.n_rows >= (1LL << 31)) return LITEVAR_ERR_UNSUPPORTED;  // 2^31 rows of 128 bytes do not fit the device
  const bool large = a.n_rows >= (1LL << 20);
  const long long rows_per_block = (kQuantThreads / 8) * (large ? 4 : 1);
  const long long blocks = (a.n_rows + rows_per_block - 1) / rows_per_block;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)blocks);
  cfg.blockDim = dim3(kQuantThreads);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = overlap ? 1 : 0;
  const cudaError_t e = large ? cudaLaunchKernelEx(&cfg, quant_rows_kernel<4>, a)
                              : cudaLaunchKernelEx(&cfg, quant_rows_kernel<1>, a);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return LITEVAR_ERR_CUDA;
  }
  return LITEVAR_OK;
}

}  // namespace

}  // namespace litevar

using namespace litevar;

extern "C" litevar_status_t litevar_quantize_rows(const void* x, const litevar_strides_t* sx, int32_t batch,
                                                  int32_t n_heads, int32_t n_tokens, int32_t head_dim, int32_t bits,
                                                  void* x_dq, const litevar_strides_t* sdq, int8_t* codes,
                                                  float* scale, float* zero, void* stream_) {
  if (!x || !quant_strides_ok(sx) || batch < 1 || n_heads < 1 || n_tokens < 1 || bits < 2 || bits > 8)
    return LITEVAR_ERR_INVALID_ARG;
  if (head_dim != kHeadDim) return LITEVAR_ERR_UNSUPPORTED;
  if (x_dq && !quant_strides_ok(sdq)) return LITEVAR_ERR_INVALID_ARG;
  if (((uintptr_t)x | (uintptr_t)x_dq) & 15) return LITEVAR_ERR_INVALID_ARG;
  if (((uintptr_t)codes & 7) || ((uintptr_t)scale & 3) || ((uintptr_t)zero & 3)) return LITEVAR_ERR_INVALID_ARG;
  QuantArgs a = {};
  a.t[0].x = static_cast<const uint16_t*>(x);
  a.t[0].dq = static_cast<uint16_t*>(x_dq);
  a.t[0].x_sb = sx->batch; a.t[0].x_sh = sx->head; a.t[0].x_st = sx->token;
  if (x_dq) { a.t[0].d_sb = sdq->batch; a.t[0].d_sh = sdq->head; a.t[0].d_st = sdq->token; }
  a.t[0].n_tokens = n_tokens;
  a.t[0].first_row = 0;
  a.n_tensors = 1;
  a.n_heads = n_heads;
  a.n_rows = (long long)batch * n_heads * n_tokens;
  a.codes = codes; a.scale = scale; a.zero = zero;
  return launch_quant(a, bits, false, static_cast<cudaStream_t>(stream_));
}

extern "C" litevar_status_t litevar_quantize_qkv(void* q, const litevar_strides_t* sq, int32_t n_q_tokens, void* k,
                                                 const litevar_strides_t* sk, void* v, const litevar_strides_t* sv,
                                                 int32_t n_kv_tokens, int32_t batch, int32_t n_heads,
                                                 int32_t head_dim, int32_t bits, void* stream_) {
  if (!q || !k || !v || !quant_strides_ok(sq) || !quant_strides_ok(sk) || !quant_strides_ok(sv) || batch < 1 ||
      n_heads < 1 || n_q_tokens < 1 || n_kv_tokens < 1 || bits < 2 || bits > 8)
    return LITEVAR_ERR_INVALID_ARG;
  if (head_dim != kHeadDim) return LITEVAR_ERR_UNSUPPORTED;
  if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v) & 15) return LITEVAR_ERR_INVALID_ARG;
  QuantArgs a = {};
  void* ptr[3] = {q, k, v};
  const litevar_strides_t* st[3] = {sq, sk, sv};
  const int32_t tokens[3] = {n_q_tokens, n_kv_tokens, n_kv_tokens};
  long long first = 0;
  for (int i = 0; i < 3; ++i) {
    a.t[i].x = static_cast<const uint16_t*>(ptr[i]);
    a.t[i].dq = static_cast<uint16_t*>(ptr[i]);
    a.t[i].x_sb = a.t[i].d_sb = st[i]->batch;
    a.t[i].x_sh = a.t[i].d_sh = st[i]->head;
    a.t[i].x_st = a.t[i].d_st = st[i]->token;
    a.t[i].n_tokens = tokens[i];
    a.t[i].first_row = first;
    first += (long long)batch * n_heads * tokens[i];
  }
  a.n_tensors = 3;
  a.n_heads = n_heads;
  a.n_rows = first;
  return launch_quant(a, bits, true, static_cast<cudaStream_t>(stream_));
}
