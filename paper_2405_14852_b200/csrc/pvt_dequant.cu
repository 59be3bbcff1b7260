// dequantize_weights (Algorithm 3, first line): W_hat = s_row * sum_m C_m[b_m] for
// every weight group.  Streaming kernel, persistent grid: two threads per group (four
// weights each), four half-groups in flight per thread, codes read coalesced,
// codewords gathered from the L2-resident codebook (small codebooks are first copied
// to shared memory), every store instruction of a warp covers whole 32-byte sectors.
//
// Arithmetic per element, binary32, each step rounded once: v = c1 (+ c2);
// w = s * v; fp16 output = round-to-nearest-even of w.
#include <cuda_fp16.h>

#include "pvt_internal.h"

namespace pvt {
namespace {

constexpr int kDqThreads = 256;
constexpr int kDqUnroll = 4;          // half-groups in flight per thread
constexpr int kDqSmemCodewords = 512;  // M*K up to this many codewords are staged in shared memory

// elements 4*half .. 4*half+3 of one codeword of 4*PARTS elements, widened to binary32
template <bool CB_F16, int PARTS>
__device__ __forceinline__ float4 load_half_codeword(const void* book, uint32_t code, uint32_t half) {
  if (CB_F16) {
    const uint2 raw = *(reinterpret_cast<const uint2*>(book) + PARTS * (size_t)code + half);
    const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
    const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
    return make_float4(lo.x, lo.y, hi.x, hi.y);
  } else {
    return *(reinterpret_cast<const float4*>(book) + PARTS * (size_t)code + half);
  }
}

// Two threads per group, four elements each: a warp then writes 512 (fp32) or 256 (fp16)
// contiguous bytes per store instruction, i.e. whole 32-byte sectors.
// (PARTS threads per group: 2 for groups of 8 weights, 4 for groups of 16.)
template <int M, bool CB_F16, bool CODE_U16, bool OUT_F16, bool SMEM_BOOK, int PARTS>
__global__ void __launch_bounds__(kDqThreads) dequant_kernel(const void* __restrict__ codebooks,
                                                              const void* __restrict__ codes,
                                                              const float* __restrict__ scale, uint64_t G,
                                                              FastDiv gpr, uint32_t K, void* __restrict__ W_hat,
                                                              uint32_t* status) {
  constexpr int kCwBytes = (CB_F16 ? 8 : 16) * PARTS;
  __shared__ __align__(16) unsigned char sh_book[SMEM_BOOK ? kDqSmemCodewords * kCwBytes : 16];
  const void* book = codebooks;
  if (SMEM_BOOK) {
    const uint4* src = reinterpret_cast<const uint4*>(codebooks);
    uint4* dst = reinterpret_cast<uint4*>(sh_book);
    const int n16 = M * K * kCwBytes / 16;
    for (int i = threadIdx.x; i < n16; i += kDqThreads) dst[i] = src[i];
    __syncthreads();
    book = sh_book;
  }
  // kDqUnroll half-groups per thread and iteration, a block apart, all their loads issued
  // before the first use: the code -> codeword -> store chain of one group is two
  // dependent memory round trips, so several must be in flight per thread
  const uint64_t H = (uint64_t)PARTS * G;
  const uint64_t stride = (uint64_t)gridDim.x * (kDqThreads * kDqUnroll);
  for (uint64_t base = (uint64_t)blockIdx.x * (kDqThreads * kDqUnroll); base < H; base += stride) {
    uint32_t b[kDqUnroll][M];
    bool bad = false;
#pragma unroll
    for (int u = 0; u < kDqUnroll; ++u) {
      const uint64_t h = base + (uint64_t)u * kDqThreads + threadIdx.x;
      const uint32_t j = (uint32_t)(h / PARTS);
#pragma unroll
      for (int m = 0; m < M; ++m) b[u][m] = 0;
      if (h < H) {
        if (CODE_U16) {
          const uint16_t* c = reinterpret_cast<const uint16_t*>(codes) + (size_t)j * M;
#pragma unroll
          for (int m = 0; m < M; ++m) b[u][m] = __ldg(c + m);
        } else if (M == 2) {
          const uint16_t both = __ldg(reinterpret_cast<const uint16_t*>(codes) + j);  // two adjacent bytes
          b[u][0] = both & 0xffu;
          b[u][M - 1] = both >> 8;
        } else {
          const uint8_t* c = reinterpret_cast<const uint8_t*>(codes) + (size_t)j * M;
#pragma unroll
          for (int m = 0; m < M; ++m) b[u][m] = __ldg(c + m);
        }
#pragma unroll
        for (int m = 0; m < M; ++m) {
          if (b[u][m] >= K) {
            bad = true;
            b[u][m] = 0;
          }
        }
      }
    }
    if (bad && status) atomicOr(status, PVT_DEV_BAD_CODE);
    float4 v[kDqUnroll];
    float s[kDqUnroll];
#pragma unroll
    for (int u = 0; u < kDqUnroll; ++u) {
      const uint64_t h = base + (uint64_t)u * kDqThreads + threadIdx.x;
      const uint32_t j = (uint32_t)(h / PARTS), half = (uint32_t)h & (uint32_t)(PARTS - 1);
      v[u] = load_half_codeword<CB_F16, PARTS>(book, b[u][0], half);
#pragma unroll
      for (int m = 1; m < M; ++m) {  // codebooks added left to right, each sum rounded once
        const float4 v2 = load_half_codeword<CB_F16, PARTS>(book, m * K + b[u][m], half);
        v[u].x = __fadd_rn(v[u].x, v2.x);
        v[u].y = __fadd_rn(v[u].y, v2.y);
        v[u].z = __fadd_rn(v[u].z, v2.z);
        v[u].w = __fadd_rn(v[u].w, v2.w);
      }
      s[u] = h < H ? __ldg(scale + fast_div(j, gpr)) : 0.0f;  // row of group j (G < 2^32)
    }
#pragma unroll
    for (int u = 0; u < kDqUnroll; ++u) {
      const uint64_t h = base + (uint64_t)u * kDqThreads + threadIdx.x;
      if (h >= H) continue;
      const float4 w = make_float4(__fmul_rn(s[u], v[u].x), __fmul_rn(s[u], v[u].y), __fmul_rn(s[u], v[u].z),
                                   __fmul_rn(s[u], v[u].w));
      if (OUT_F16) {
        const __half2 lo = __floats2half2_rn(w.x, w.y), hi = __floats2half2_rn(w.z, w.w);
        __stcs(reinterpret_cast<uint2*>(W_hat) + h,
               make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi)));
      } else {
        __stcs(reinterpret_cast<float4*>(W_hat) + h, w);
      }
    }
  }
}

template <int M, bool CB_F16, bool CODE_U16, bool OUT_F16, int PARTS = 2>
cudaError_t launch_t(const pvt_layer& L, uint64_t G, void* W_hat, uint32_t* status, int sm_count,
                     cudaStream_t stream) {
  const bool smem_book = (uint32_t)M * (uint32_t)L.codebook_size * (PARTS / 2) <= (uint32_t)kDqSmemCodewords;
  // persistent grid: as many blocks as are resident at once
  int per_sm = 0;
  cudaError_t oe = smem_book ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(
                                   &per_sm, dequant_kernel<M, CB_F16, CODE_U16, OUT_F16, true, PARTS>, kDqThreads, 0)
                             : cudaOccupancyMaxActiveBlocksPerMultiprocessor(
                                   &per_sm, dequant_kernel<M, CB_F16, CODE_U16, OUT_F16, false, PARTS>, kDqThreads, 0);
  if (oe != cudaSuccess) return oe;
  if (per_sm < 1) per_sm = 1;
  const uint64_t per_block = (uint64_t)kDqThreads * kDqUnroll;
  const uint64_t want = (PARTS * G + per_block - 1) / per_block;
  const uint64_t cap = (uint64_t)sm_count * (uint64_t)per_sm;
  const unsigned blocks = (unsigned)(want < cap ? want : cap);
  const FastDiv gpr = make_fast_div((uint32_t)(L.cols / (4 * PARTS)));  // groups per row
  const uint32_t K = (uint32_t)L.codebook_size;
  if (smem_book)
    dequant_kernel<M, CB_F16, CODE_U16, OUT_F16, true, PARTS>
        <<<blocks, kDqThreads, 0, stream>>>(L.codebooks, L.codes, L.scale, G, gpr, K, W_hat, status);
  else
    dequant_kernel<M, CB_F16, CODE_U16, OUT_F16, false, PARTS>
        <<<blocks, kDqThreads, 0, stream>>>(L.codebooks, L.codes, L.scale, G, gpr, K, W_hat, status);
  return cudaGetLastError();
}

template <int M, bool CB_F16, bool CODE_U16>
cudaError_t launch_o(const pvt_layer& L, uint64_t G, void* W_hat, int32_t out_dtype, uint32_t* status,
                     int sm_count, cudaStream_t stream) {
  return out_dtype == PVT_F16 ? launch_t<M, CB_F16, CODE_U16, true>(L, G, W_hat, status, sm_count, stream)
                              : launch_t<M, CB_F16, CODE_U16, false>(L, G, W_hat, status, sm_count, stream);
}

template <int M, bool CB_F16>
cudaError_t launch_c(const pvt_layer& L, uint64_t G, void* W_hat, int32_t out_dtype, uint32_t* status,
                     int sm_count, cudaStream_t stream) {
  return L.code_dtype == PVT_U16 ? launch_o<M, CB_F16, true>(L, G, W_hat, out_dtype, status, sm_count, stream)
                                 : launch_o<M, CB_F16, false>(L, G, W_hat, out_dtype, status, sm_count, stream);
}

}  // namespace

cudaError_t launch_dequant(const pvt_layer& L, uint64_t G, void* W_hat, int32_t out_dtype, uint32_t* status,
                           int sm_count, cudaStream_t stream) {
  timing_begin(kKernDequant, stream);
  cudaError_t err;
  const bool f16 = L.codebook_dtype == PVT_F16;
  if (L.group_dim == 16) {  // groups of 16 weights: one codebook
    const bool u16 = L.code_dtype == PVT_U16, o16 = out_dtype == PVT_F16;
#define PVT_DQ16(CB, CU, OF) launch_t<1, CB, CU, OF, 4>(L, G, W_hat, status, sm_count, stream)
    if (f16)
      err = u16 ? (o16 ? PVT_DQ16(true, true, true) : PVT_DQ16(true, true, false))
                : (o16 ? PVT_DQ16(true, false, true) : PVT_DQ16(true, false, false));
    else
      err = u16 ? (o16 ? PVT_DQ16(false, true, true) : PVT_DQ16(false, true, false))
                : (o16 ? PVT_DQ16(false, false, true) : PVT_DQ16(false, false, false));
#undef PVT_DQ16
    count_launches(1);
    timing_end(kKernDequant, stream);
    return err;
  }
  switch (L.num_codebooks) {
    case 1:
      err = f16 ? launch_c<1, true>(L, G, W_hat, out_dtype, status, sm_count, stream)
                : launch_c<1, false>(L, G, W_hat, out_dtype, status, sm_count, stream);
      break;
    case 2:
      err = f16 ? launch_c<2, true>(L, G, W_hat, out_dtype, status, sm_count, stream)
                : launch_c<2, false>(L, G, W_hat, out_dtype, status, sm_count, stream);
      break;
    case 3:
      err = f16 ? launch_c<3, true>(L, G, W_hat, out_dtype, status, sm_count, stream)
                : launch_c<3, false>(L, G, W_hat, out_dtype, status, sm_count, stream);
      break;
    default:
      err = f16 ? launch_c<4, true>(L, G, W_hat, out_dtype, status, sm_count, stream)
                : launch_c<4, false>(L, G, W_hat, out_dtype, status, sm_count, stream);
      break;
  }
  count_launches(1);
  timing_end(kKernDequant, stream);
  return err;
}

}  // namespace pvt
