// Exhaustive nearest-codeword search for groups of 16 weights and one codebook (Appendix J: the representations
// with group size 16 and one codebook of up to 2^16 codewords).  First version: every distance is the binary64
// value the decision is defined on, sum_i (t_i - c_i)^2 with the terms added in element order, so the result is
// the argmin of (distance, code) with no filter and no rescoring.
//
// A block owns 16 targets (two per warp, in registers as binary64) and streams the codebook through shared memory
// in chunks of 128 codewords widened to binary64; a lane scores the codewords lane, lane+32, ... of a chunk against
// its warp's two targets.  Cost per target: K * 48 binary64 operations and K * 64 bytes of shared-memory reads.
#include <cuda_fp16.h>

#include "pvt_internal.h"

namespace pvt {
namespace {

constexpr int kG16Threads = 256;
constexpr int kG16PerWarp = 2;
constexpr int kG16PerBlock = (kG16Threads / 32) * kG16PerWarp;  // 16 targets
constexpr int kG16Chunk = 128;                                  // codewords per staged chunk
constexpr int kG16Row = 17;                                     // doubles per staged codeword (16 + 1 against bank conflicts)
constexpr long long kInf = 0x7ff0000000000000ll;

struct G16Params {
  const float* W;
  const float* g;
  const float* scale;
  const void* book;
  void* codes;
  const uint32_t* idx;
  uint64_t k, G;
  uint32_t gpr, K;
  float eta;
  float* err_out;
  uint32_t* status;
};

template <bool CB_F16, bool CODE_U16>
__global__ void __launch_bounds__(kG16Threads) encode_g16_kernel(const G16Params p) {
  __shared__ double chunk[kG16Chunk * kG16Row];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t K = p.K;

  // the two targets of this warp (Eq. 8 in the scaled space: one fma and one division per element, binary32)
  double t[kG16PerWarp][16];
  uint32_t jj[kG16PerWarp];
  bool have[kG16PerWarp];
#pragma unroll
  for (int u = 0; u < kG16PerWarp; ++u) {
    const uint64_t n = (uint64_t)blockIdx.x * kG16PerBlock + warp * kG16PerWarp + u;
    have[u] = false;
    jj[u] = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) t[u][i] = 0.0;
    if (n < p.k) {
      const uint32_t j = __ldg(p.idx + n);
      if (j < p.G) {
        have[u] = true;
        jj[u] = j;
        const float4* W4 = reinterpret_cast<const float4*>(p.W) + 4 * (size_t)j;
        const float4* g4 = reinterpret_cast<const float4*>(p.g) + 4 * (size_t)j;
        const float s = __ldg(p.scale + j / p.gpr), ne = -p.eta;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float4 w = __ldg(W4 + q), gg = __ldg(g4 + q);
          t[u][4 * q + 0] = (double)__fdiv_rn(__fmaf_rn(ne, gg.x, w.x), s);
          t[u][4 * q + 1] = (double)__fdiv_rn(__fmaf_rn(ne, gg.y, w.y), s);
          t[u][4 * q + 2] = (double)__fdiv_rn(__fmaf_rn(ne, gg.z, w.z), s);
          t[u][4 * q + 3] = (double)__fdiv_rn(__fmaf_rn(ne, gg.w, w.w), s);
        }
      } else if (lane == 0) {
        atomicOr(p.status, PVT_DEV_BAD_INDEX);
      }
    }
  }
  double best_d[kG16PerWarp];
  uint32_t best_c[kG16PerWarp];
#pragma unroll
  for (int u = 0; u < kG16PerWarp; ++u) {
    best_d[u] = __longlong_as_double(kInf);
    best_c[u] = 0xffffffffu;
  }

  for (uint32_t c0 = 0; c0 < K; c0 += kG16Chunk) {
    __syncthreads();  // the previous chunk has been read by every warp
    // stage codewords c0 .. c0+127 widened to binary64: four elements per thread and step
    for (int item = threadIdx.x; item < kG16Chunk * 4; item += kG16Threads) {
      const uint32_t row = item >> 2, quarter = item & 3, code = c0 + row;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (code < K) {
        if (CB_F16) {
          const uint2 raw = __ldg(reinterpret_cast<const uint2*>(p.book) + 4 * (size_t)code + quarter);
          const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
          const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
          v = make_float4(lo.x, lo.y, hi.x, hi.y);
        } else {
          v = __ldg(reinterpret_cast<const float4*>(p.book) + 4 * (size_t)code + quarter);
        }
      }
      double* dst = &chunk[row * kG16Row + 4 * quarter];
      dst[0] = (double)v.x;
      dst[1] = (double)v.y;
      dst[2] = (double)v.z;
      dst[3] = (double)v.w;
    }
    __syncthreads();
#pragma unroll 1
    for (int r = lane; r < kG16Chunk; r += 32) {
      const uint32_t code = c0 + r;
      if (code >= K) break;
      const double* c = &chunk[r * kG16Row];
      double d[kG16PerWarp];
#pragma unroll
      for (int u = 0; u < kG16PerWarp; ++u) d[u] = 0.0;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const double ci = c[i];
#pragma unroll
        for (int u = 0; u < kG16PerWarp; ++u) {
          const double e = __dsub_rn(t[u][i], ci);
          d[u] = __dadd_rn(d[u], __dmul_rn(e, e));
        }
      }
#pragma unroll
      for (int u = 0; u < kG16PerWarp; ++u)
        if (d[u] < best_d[u]) {  // codes ascend within a lane: equal distances keep the lower code
          best_d[u] = d[u];
          best_c[u] = code;
        }
    }
  }

  // warp-wide argmin of (distance, code); distances are >= 0, so their bits order like u64
#pragma unroll
  for (int u = 0; u < kG16PerWarp; ++u) {
    const uint64_t bits = (uint64_t)__double_as_longlong(best_d[u]);
    const uint32_t hi = (uint32_t)(bits >> 32), lo = (uint32_t)bits;
    const uint32_t mhi = __reduce_min_sync(0xffffffffu, hi);
    const uint32_t mlo = __reduce_min_sync(0xffffffffu, hi == mhi ? lo : 0xffffffffu);
    const uint32_t mc = __reduce_min_sync(0xffffffffu, (hi == mhi && lo == mlo) ? best_c[u] : 0xffffffffu);
    if (lane == 0 && have[u]) {
      if (mc < K) {
        if (CODE_U16)
          reinterpret_cast<uint16_t*>(p.codes)[jj[u]] = (uint16_t)mc;
        else
          reinterpret_cast<uint8_t*>(p.codes)[jj[u]] = (uint8_t)mc;
        const uint64_t n = (uint64_t)blockIdx.x * kG16PerBlock + warp * kG16PerWarp + u;
        if (p.err_out) p.err_out[n] = (float)__longlong_as_double((long long)(((uint64_t)mhi << 32) | mlo));
      } else {
        atomicOr(p.status, PVT_DEV_INTERNAL);  // non-finite target: no distance compares below infinity
      }
    }
  }
}

}  // namespace

cudaError_t launch_encode_g16(const pvt_layer& L, uint64_t G, const uint32_t* idx, uint64_t k, float* err_out,
                              void* ws, cudaStream_t stream) {
  G16Params p;
  p.W = L.W;
  p.g = L.g;
  p.scale = L.scale;
  p.book = L.codebooks;
  p.codes = L.codes;
  p.idx = idx;
  p.k = k;
  p.G = G;
  p.gpr = (uint32_t)(L.cols / 16);
  p.K = (uint32_t)L.codebook_size;
  p.eta = L.eta;
  p.err_out = err_out;
  p.status = static_cast<uint32_t*>(ws);
  const unsigned blocks = (unsigned)((k + kG16PerBlock - 1) / kG16PerBlock);
  const bool f16 = L.codebook_dtype == PVT_F16, u16 = L.code_dtype == PVT_U16;
  timing_begin(kKernEncodeMain, stream);
  if (f16) {
    if (u16)
      encode_g16_kernel<true, true><<<blocks, kG16Threads, 0, stream>>>(p);
    else
      encode_g16_kernel<true, false><<<blocks, kG16Threads, 0, stream>>>(p);
  } else {
    if (u16)
      encode_g16_kernel<false, true><<<blocks, kG16Threads, 0, stream>>>(p);
    else
      encode_g16_kernel<false, false><<<blocks, kG16Threads, 0, stream>>>(p);
  }
  count_launches(1);
  timing_end(kKernEncodeMain, stream);
  return cudaGetLastError();
}

}  // namespace pvt
