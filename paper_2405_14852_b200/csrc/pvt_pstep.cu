// The part of the P step that shares its inputs with the V step (Algorithm 3, P-step lines:
// grad_codebooks = backprop(grad_phi); codebooks = adam(grad_codebooks); Section 3.4 and Appendix J for Adam
// and its betas).
//
// backprop is the chain rule through dequantize_weights, W_hat[r, 8c + i] = s_r * v_{j,i} with
// v_j = sum_m C_m[b_{j,m}] (the binary32 sum that dequantisation forms):
//     grad_codebooks[m][kappa][i] = sum over groups j with b_{j,m} = kappa of  s_{r(j)} * g[j][i]
//     grad_scale[r]               = sum over groups j of row r and over i of   g[j][i] * v_{j,i}
// Every product of two binary32 numbers is exact in binary64 and the sums are accumulated in binary64 with
// atomic adds, so the result differs from a sequential sum only by the order of binary64 roundings.
//
// One streaming pass over g (two threads per group, 512 contiguous bytes per warp load).  Small codebooks
// (M K <= 512 codewords) are accumulated in shared memory per block and flushed once; large ones go straight
// to the L2 with one reduction per element.  Scale gradients are summed over a warp first when the warp
// lies inside one row.
#include <cuda_fp16.h>

#include "pvt_internal.h"

namespace pvt {
namespace {

constexpr int kPsThreads = 256;
constexpr int kPsSmemCodewords = 512;

// elements 4*half .. 4*half+3 of a codeword of 4*PARTS elements (PARTS = 2 for groups of 8 weights, 4 for 16)
template <bool CB_F16, int PARTS = 2>
__device__ __forceinline__ float4 half_codeword(const void* book, uint32_t code, uint32_t half) {
  if (CB_F16) {
    const uint2 raw = __ldg(reinterpret_cast<const uint2*>(book) + PARTS * (size_t)code + half);
    const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
    const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
    return make_float4(lo.x, lo.y, hi.x, hi.y);
  } else {
    return __ldg(reinterpret_cast<const float4*>(book) + PARTS * (size_t)code + half);
  }
}

__device__ __forceinline__ void red_add_f64(double* p, double v) {
  asm volatile("red.global.add.f64 [%0], %1;" ::"l"(p), "d"(v) : "memory");
}

template <int M, bool CB_F16, bool CODE_U16, bool SMEM_ACC, int PARTS = 2>
__global__ void __launch_bounds__(kPsThreads) pstep_grad_kernel(const float* __restrict__ g,
                                                                 const float* __restrict__ scale,
                                                                 const void* __restrict__ codes,
                                                                 const void* __restrict__ codebooks, uint64_t G,
                                                                 uint32_t gpr, uint32_t K,
                                                                 double* __restrict__ grad_books,
                                                                 double* __restrict__ grad_scale, uint32_t* status) {
  __shared__ double sh_acc[SMEM_ACC ? kPsSmemCodewords * 8 : 1];
  if (SMEM_ACC) {
    for (uint32_t i = threadIdx.x; i < (uint32_t)M * K * 8; i += kPsThreads) sh_acc[i] = 0.0;
    __syncthreads();
  }
  const uint64_t H = (uint64_t)PARTS * G;  // PARTS threads per group, four weights each
  const float4* g4 = reinterpret_cast<const float4*>(g);
  const int lane = threadIdx.x & 31;
  for (uint64_t h0 = (uint64_t)blockIdx.x * kPsThreads; h0 < H; h0 += (uint64_t)gridDim.x * kPsThreads) {
    const uint64_t h = h0 + threadIdx.x;
    const bool valid = h < H;
    const uint32_t j = (uint32_t)(h / PARTS), half = (uint32_t)h & (uint32_t)(PARTS - 1);
    uint32_t row = 0xffffffffu;
    double ds = 0.0;
    if (valid) {
      const float4 gv = __ldcs(g4 + h);
      row = j / gpr;
      const float s = __ldg(scale + row);
      uint32_t b[M];
      if (CODE_U16) {
        const uint16_t* c = reinterpret_cast<const uint16_t*>(codes) + (size_t)j * M;
#pragma unroll
        for (int m = 0; m < M; ++m) b[m] = __ldg(c + m);
      } else if (M == 2) {
        const uint16_t both = __ldg(reinterpret_cast<const uint16_t*>(codes) + j);
        b[0] = both & 0xffu;
        b[M - 1] = both >> 8;
      } else {
        const uint8_t* c = reinterpret_cast<const uint8_t*>(codes) + (size_t)j * M;
#pragma unroll
        for (int m = 0; m < M; ++m) b[m] = __ldg(c + m);
      }
      bool bad = false;
#pragma unroll
      for (int m = 0; m < M; ++m) {
        if (b[m] >= K) {
          bad = true;
          b[m] = 0;
        }
      }
      if (bad) {
        if (status) atomicOr(status, PVT_DEV_BAD_CODE);
      } else {
        // codebook gradients: s * g, exact in binary64
        const double sd = (double)s;
        const double p0 = sd * (double)gv.x, p1 = sd * (double)gv.y, p2 = sd * (double)gv.z, p3 = sd * (double)gv.w;
#pragma unroll
        for (int m = 0; m < M; ++m) {
          const size_t at = ((size_t)m * K + b[m]) * (4 * PARTS) + half * 4;
          if (SMEM_ACC) {
            atomicAdd(&sh_acc[at], p0);
            atomicAdd(&sh_acc[at + 1], p1);
            atomicAdd(&sh_acc[at + 2], p2);
            atomicAdd(&sh_acc[at + 3], p3);
          } else {
            red_add_f64(grad_books + at, p0);
            red_add_f64(grad_books + at + 1, p1);
            red_add_f64(grad_books + at + 2, p2);
            red_add_f64(grad_books + at + 3, p3);
          }
        }
        if (grad_scale) {
          float4 v = half_codeword<CB_F16, PARTS>(codebooks, b[0], half);
#pragma unroll
          for (int m = 1; m < M; ++m) {
            const float4 v2 = half_codeword<CB_F16, PARTS>(codebooks, m * K + b[m], half);
            v.x = __fadd_rn(v.x, v2.x);
            v.y = __fadd_rn(v.y, v2.y);
            v.z = __fadd_rn(v.z, v2.z);
            v.w = __fadd_rn(v.w, v2.w);
          }
          ds = (double)gv.x * (double)v.x;
          ds = __dadd_rn(ds, (double)gv.y * (double)v.y);
          ds = __dadd_rn(ds, (double)gv.z * (double)v.z);
          ds = __dadd_rn(ds, (double)gv.w * (double)v.w);
        }
      }
    }
    if (grad_scale) {
      // a warp that lies inside one row adds its 32 contributions with one reduction
      const uint32_t row0 = __shfl_sync(0xffffffffu, row, 0);
      if (__all_sync(0xffffffffu, row == row0)) {
#pragma unroll
        for (int o = 16; o; o >>= 1) ds = __dadd_rn(ds, __shfl_xor_sync(0xffffffffu, ds, o));
        if (lane == 0 && row0 != 0xffffffffu) red_add_f64(grad_scale + row0, ds);
      } else if (row != 0xffffffffu) {
        red_add_f64(grad_scale + row, ds);
      }
    }
  }
  if (SMEM_ACC) {
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < (uint32_t)M * K * 8; i += kPsThreads)
      if (sh_acc[i] != 0.0) red_add_f64(grad_books + i, sh_acc[i]);
  }
}


// Small codebooks with one-byte codes (M K <= 512): no floating-point atomics in the block.  A block takes tiles
// of 512 groups; per tile it stages the exact products s * g in shared memory, counting-sorts the tile's groups by
// code (integer shared-memory atomics hand out the slots), and then every accumulator (codebook, code, element)
// is owned by one thread, which adds the products of the code's groups in binary64 with plain
// additions.  The accumulators go to the L2 once per block.
constexpr int kPsTile = 512;

template <int M, bool CB_F16>
__global__ void __launch_bounds__(kPsThreads) pstep_grad_sorted_kernel(const float* __restrict__ g,
                                                                        const float* __restrict__ scale,
                                                                        const uint8_t* __restrict__ codes,
                                                                        const void* __restrict__ codebooks, uint64_t G,
                                                                        uint32_t gpr, uint32_t K,
                                                                        double* __restrict__ grad_books,
                                                                        double* __restrict__ grad_scale,
                                                                        uint32_t* status) {
  extern __shared__ __align__(16) unsigned char ps_smem[];
  double* sh_acc = reinterpret_cast<double*>(ps_smem);                       // [M*K*8]
  double* sh_p = sh_acc + (size_t)M * K * 8;                                 // [tile][8]: the exact products s * g
  uint32_t* sh_cnt = reinterpret_cast<uint32_t*>(sh_p + kPsTile * 8);        // [M][256] counts
  uint32_t* sh_start = sh_cnt + M * 256;                                     // [M][256]
  uint16_t* sh_sorted = reinterpret_cast<uint16_t*>(sh_start + M * 256);     // [M][tile]
  uint16_t* sh_slot = sh_sorted + M * kPsTile;                               // [M][tile]: slot of group in its bin
  uint8_t* sh_code = reinterpret_cast<uint8_t*>(sh_slot + M * kPsTile);      // [M][tile]

  for (uint32_t i = threadIdx.x; i < (uint32_t)M * K * 8; i += kPsThreads) sh_acc[i] = 0.0;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const float4* g4 = reinterpret_cast<const float4*>(g);
  const uint64_t n_tiles = (G + kPsTile - 1) / kPsTile;
  for (uint64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const uint64_t j0 = tile * kPsTile;
    const uint32_t n_here = (uint32_t)(G - j0 < (uint64_t)kPsTile ? G - j0 : (uint64_t)kPsTile);
    __syncthreads();  // the previous tile has been consumed
    for (uint32_t i = threadIdx.x; i < (uint32_t)M * 256; i += kPsThreads) sh_cnt[i] = 0;
    __syncthreads();
    // stage the tile: two threads per group (512 contiguous bytes per warp load); all loads of the tile are
    // issued before the first use, the pass is bound by memory latency otherwise
    constexpr int kIter = 2 * kPsTile / kPsThreads;  // 8 half-groups per thread
    float4 gv_all[kIter];
    uint32_t b_all[kIter][M];
#pragma unroll
    for (int it = 0; it < kIter; ++it) {
      const uint32_t hh = it * kPsThreads + threadIdx.x, slot = hh >> 1, half = hh & 1u;
      gv_all[it] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int m = 0; m < M; ++m) b_all[it][m] = 0;
      if (slot < n_here) {
        const uint64_t j = j0 + slot;
        gv_all[it] = __ldcs(g4 + 2 * j + half);
#pragma unroll
        for (int m = 0; m < M; ++m) b_all[it][m] = __ldg(codes + j * M + m);
      }
    }
#pragma unroll
    for (int it = 0; it < kIter; ++it) {
      const uint32_t hh = it * kPsThreads + threadIdx.x, slot = hh >> 1, half = hh & 1u;
      const uint64_t j = j0 + slot;
      uint32_t row = 0xffffffffu;
      double ds = 0.0;
      if (slot < n_here) {
        const float4 gv = gv_all[it];
        row = (uint32_t)j / gpr;
        uint32_t b[M];
        bool bad = false;
#pragma unroll
        for (int m = 0; m < M; ++m) {
          b[m] = b_all[it][m];
          if (b[m] >= K) {
            bad = true;
            b[m] = 0;
          }
        }
        {
          const double sd = bad ? 0.0 : (double)__ldg(scale + row);  // a group with a bad code contributes nothing
          double* dst = &sh_p[slot * 8 + half * 4];
          dst[0] = sd * (double)gv.x;
          dst[1] = sd * (double)gv.y;
          dst[2] = sd * (double)gv.z;
          dst[3] = sd * (double)gv.w;
        }
        if (half == 0) {
#pragma unroll
          for (int m = 0; m < M; ++m) {
            sh_code[m * kPsTile + slot] = (uint8_t)b[m];
            sh_slot[m * kPsTile + slot] = (uint16_t)atomicAdd(&sh_cnt[m * 256 + b[m]], 1u);
          }
        }
        if (bad) {
          if (status) atomicOr(status, PVT_DEV_BAD_CODE);
        } else if (grad_scale) {
          float4 v = half_codeword<CB_F16>(codebooks, b[0], half);
#pragma unroll
          for (int m = 1; m < M; ++m) {
            const float4 v2 = half_codeword<CB_F16>(codebooks, m * K + b[m], half);
            v.x = __fadd_rn(v.x, v2.x);
            v.y = __fadd_rn(v.y, v2.y);
            v.z = __fadd_rn(v.z, v2.z);
            v.w = __fadd_rn(v.w, v2.w);
          }
          ds = (double)gv.x * (double)v.x;
          ds = __dadd_rn(ds, (double)gv.y * (double)v.y);
          ds = __dadd_rn(ds, (double)gv.z * (double)v.z);
          ds = __dadd_rn(ds, (double)gv.w * (double)v.w);
        }
      }
      if (grad_scale) {
        const uint32_t row0 = __shfl_sync(0xffffffffu, row, 0);
        if (__all_sync(0xffffffffu, row == row0)) {
#pragma unroll
          for (int o = 16; o; o >>= 1) ds = __dadd_rn(ds, __shfl_xor_sync(0xffffffffu, ds, o));
          if (lane == 0 && row0 != 0xffffffffu) red_add_f64(grad_scale + row0, ds);
        } else if (row != 0xffffffffu) {
          red_add_f64(grad_scale + row, ds);
        }
      }
    }
    __syncthreads();
    // exclusive prefix of the counts per codebook: one warp per codebook, eight bins per lane
    if (warp < M) {
      uint32_t c[8], sum = 0;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        c[q] = sh_cnt[warp * 256 + lane * 8 + q];
        sum += c[q];
      }
      uint32_t incl = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
      }
      uint32_t run = incl - sum;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        sh_start[warp * 256 + lane * 8 + q] = run;
        run += c[q];
      }
    }
    __syncthreads();
#pragma unroll
    for (int m = 0; m < M; ++m)
      for (uint32_t slot = threadIdx.x; slot < n_here; slot += kPsThreads) {
        const uint32_t code = sh_code[m * kPsTile + slot];
        sh_sorted[m * kPsTile + sh_start[m * 256 + code] + sh_slot[m * kPsTile + slot]] = (uint16_t)slot;
      }
    __syncthreads();
    // every accumulator (codebook, code, element) is owned by one thread: plain binary64 additions over the
    // code's groups; eight adjacent threads share a code, so its group list is a broadcast load
#pragma unroll
    for (int m = 0; m < M; ++m)
      for (uint32_t bin = threadIdx.x; bin < K * 8; bin += kPsThreads) {
        const uint32_t code = bin >> 3, e = bin & 7u;
        const uint32_t cnt = sh_cnt[m * 256 + code];
        if (cnt == 0) continue;
        const uint16_t* list = &sh_sorted[m * kPsTile + sh_start[m * 256 + code]];
        double acc = 0.0;
        for (uint32_t i = 0; i < cnt; ++i) acc = __dadd_rn(acc, sh_p[(uint32_t)list[i] * 8 + e]);
        sh_acc[((size_t)m * K + code) * 8 + e] += acc;
      }
  }
  __syncthreads();
  for (uint32_t i = threadIdx.x; i < (uint32_t)M * K * 8; i += kPsThreads)
    if (sh_acc[i] != 0.0) red_add_f64(grad_books + i, sh_acc[i]);
}

template <int M, bool CB_F16>
cudaError_t launch_grad_sorted(const pvt_layer& L, uint64_t G, double* grad_books, double* grad_scale, uint32_t* status,
                               int sm_count, cudaStream_t stream) {
  const uint32_t gpr = (uint32_t)(L.cols / kGroupDim), K = (uint32_t)L.codebook_size;
  const size_t smem = sizeof(double) * M * K * 8 + sizeof(double) * kPsTile * 8 + sizeof(uint32_t) * M * 512 +
                      sizeof(uint16_t) * M * kPsTile * 2 + (size_t)M * kPsTile;
  cudaError_t e = cudaFuncSetAttribute(pstep_grad_sorted_kernel<M, CB_F16>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, pstep_grad_sorted_kernel<M, CB_F16>, kPsThreads, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) per_sm = 1;
  const uint64_t tiles = (G + kPsTile - 1) / kPsTile, cap = (uint64_t)sm_count * per_sm;
  pstep_grad_sorted_kernel<M, CB_F16><<<(unsigned)(tiles < cap ? tiles : cap), kPsThreads, smem, stream>>>(
      L.g, L.scale, static_cast<const uint8_t*>(L.codes), L.codebooks, G, gpr, K, grad_books, grad_scale, status);
  return cudaGetLastError();
}

template <int M, bool CB_F16, bool CODE_U16>
cudaError_t launch_grad(const pvt_layer& L, uint64_t G, double* grad_books, double* grad_scale, uint32_t* status,
                        int sm_count, cudaStream_t stream) {
  const uint32_t gpr = (uint32_t)(L.cols / kGroupDim), K = (uint32_t)L.codebook_size;
  if (L.group_dim == 16) {  // groups of 16 weights (one codebook): four threads per group, reductions in the L2
    const uint64_t want16 = (4 * G + kPsThreads - 1) / kPsThreads, cap16 = (uint64_t)sm_count * 8;
    pstep_grad_kernel<M, CB_F16, CODE_U16, false, 4><<<(unsigned)(want16 < cap16 ? want16 : cap16), kPsThreads, 0, stream>>>(
        L.g, L.scale, L.codes, L.codebooks, G, (uint32_t)(L.cols / 16), K, grad_books, grad_scale, status);
    return cudaGetLastError();
  }
  const bool smem_acc = (uint32_t)M * K <= (uint32_t)kPsSmemCodewords;
  if (smem_acc && !CODE_U16) return launch_grad_sorted<M, CB_F16>(L, G, grad_books, grad_scale, status, sm_count, stream);
  const uint64_t want = (2 * G + kPsThreads - 1) / kPsThreads;
  const uint64_t cap = (uint64_t)sm_count * (smem_acc ? 4 : 8);
  const unsigned blocks = (unsigned)(want < cap ? want : cap);
  if (smem_acc)
    pstep_grad_kernel<M, CB_F16, CODE_U16, true><<<blocks, kPsThreads, 0, stream>>>(
        L.g, L.scale, L.codes, L.codebooks, G, gpr, K, grad_books, grad_scale, status);
  else
    pstep_grad_kernel<M, CB_F16, CODE_U16, false><<<blocks, kPsThreads, 0, stream>>>(
        L.g, L.scale, L.codes, L.codebooks, G, gpr, K, grad_books, grad_scale, status);
  return cudaGetLastError();
}

// One Adam update, binary32, each operation rounded once, in the order stated in pvt.h.
__global__ void __launch_bounds__(256) adam_kernel(float* __restrict__ param, __half* __restrict__ param_f16,
                                                    const double* __restrict__ grad, float* __restrict__ exp_avg,
                                                    float* __restrict__ exp_avg_sq, uint64_t n, float lr, float beta1,
                                                    float beta2, float eps, float bias1, float bias2) {
  const float omb1 = __fsub_rn(1.0f, beta1), omb2 = __fsub_rn(1.0f, beta2);
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
    const float gr = __double2float_rn(grad[i]);
    const float m = __fmaf_rn(beta1, exp_avg[i], __fmul_rn(omb1, gr));
    const float v = __fmaf_rn(beta2, exp_avg_sq[i], __fmul_rn(__fmul_rn(omb2, gr), gr));
    exp_avg[i] = m;
    exp_avg_sq[i] = v;
    const float num = __fmul_rn(lr, __fdiv_rn(m, bias1));
    const float den = __fadd_rn(__fsqrt_rn(__fdiv_rn(v, bias2)), eps);
    const float p = __fsub_rn(param[i], __fdiv_rn(num, den));
    param[i] = p;
    if (param_f16) param_f16[i] = __float2half_rn(p);
  }
}

// Adam-normalised update direction of the V step (Section 3.4): moments as in Adam, u = (m / bias1) /
// (sqrt(v / bias2) + eps), binary32, each operation rounded once.  Four elements per thread (128-bit accesses).
__global__ void __launch_bounds__(256) adam_direction_kernel(const float4* __restrict__ grad, float4* __restrict__ exp_avg,
                                                              float4* __restrict__ exp_avg_sq, float4* __restrict__ dir,
                                                              uint64_t n4, float beta1, float beta2, float eps,
                                                              float bias1, float bias2) {
  const float omb1 = __fsub_rn(1.0f, beta1), omb2 = __fsub_rn(1.0f, beta2);
  auto one = [&](float gr, float& m, float& v) {
    m = __fmaf_rn(beta1, m, __fmul_rn(omb1, gr));
    v = __fmaf_rn(beta2, v, __fmul_rn(__fmul_rn(omb2, gr), gr));
    return __fdiv_rn(__fdiv_rn(m, bias1), __fadd_rn(__fsqrt_rn(__fdiv_rn(v, bias2)), eps));
  };
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (uint64_t)gridDim.x * blockDim.x) {
    const float4 g = __ldcs(grad + i);
    float4 m = exp_avg[i], v = exp_avg_sq[i], u;
    u.x = one(g.x, m.x, v.x);
    u.y = one(g.y, m.y, v.y);
    u.z = one(g.z, m.z, v.z);
    u.w = one(g.w, m.w, v.w);
    exp_avg[i] = m;
    exp_avg_sq[i] = v;
    dir[i] = u;
  }
}

}  // namespace

cudaError_t launch_adam_direction(const float* grad, float* exp_avg, float* exp_avg_sq, float* dir, uint64_t n,
                                  float beta1, float beta2, float eps, float bias1, float bias2, int sm_count,
                                  cudaStream_t stream) {
  timing_begin(kKernAdam, stream);
  const uint64_t n4 = n / 4, want = (n4 + 255) / 256, cap = (uint64_t)sm_count * 8;
  adam_direction_kernel<<<(unsigned)(want < cap ? want : cap), 256, 0, stream>>>(
      reinterpret_cast<const float4*>(grad), reinterpret_cast<float4*>(exp_avg), reinterpret_cast<float4*>(exp_avg_sq),
      reinterpret_cast<float4*>(dir), n4, beta1, beta2, eps, bias1, bias2);
  count_launches(1);
  timing_end(kKernAdam, stream);
  return cudaGetLastError();
}

cudaError_t launch_pstep_grad(const pvt_layer& L, uint64_t G, double* grad_books, double* grad_scale, uint32_t* status,
                              int sm_count, cudaStream_t stream) {
  cudaError_t err = cudaMemsetAsync(grad_books, 0,
                                    sizeof(double) * (size_t)L.num_codebooks * (size_t)L.codebook_size * (size_t)L.group_dim, stream);
  if (err != cudaSuccess) return err;
  if (grad_scale && (err = cudaMemsetAsync(grad_scale, 0, sizeof(double) * (size_t)L.rows, stream)) != cudaSuccess)
    return err;
  timing_begin(kKernPstepGrad, stream);
  const bool f16 = L.codebook_dtype == PVT_F16, u16 = L.code_dtype == PVT_U16;
  if (L.num_codebooks == 1) {
    if (f16)
      err = u16 ? launch_grad<1, true, true>(L, G, grad_books, grad_scale, status, sm_count, stream)
                : launch_grad<1, true, false>(L, G, grad_books, grad_scale, status, sm_count, stream);
    else
      err = u16 ? launch_grad<1, false, true>(L, G, grad_books, grad_scale, status, sm_count, stream)
                : launch_grad<1, false, false>(L, G, grad_books, grad_scale, status, sm_count, stream);
  } else if (L.num_codebooks == 2) {
    if (f16)
      err = u16 ? launch_grad<2, true, true>(L, G, grad_books, grad_scale, status, sm_count, stream)
                : launch_grad<2, true, false>(L, G, grad_books, grad_scale, status, sm_count, stream);
    else
      err = u16 ? launch_grad<2, false, true>(L, G, grad_books, grad_scale, status, sm_count, stream)
                : launch_grad<2, false, false>(L, G, grad_books, grad_scale, status, sm_count, stream);
  } else if (L.num_codebooks == 3) {  // three and four codebooks: one-byte codes
    err = f16 ? launch_grad<3, true, false>(L, G, grad_books, grad_scale, status, sm_count, stream)
              : launch_grad<3, false, false>(L, G, grad_books, grad_scale, status, sm_count, stream);
  } else {
    err = f16 ? launch_grad<4, true, false>(L, G, grad_books, grad_scale, status, sm_count, stream)
              : launch_grad<4, false, false>(L, G, grad_books, grad_scale, status, sm_count, stream);
  }
  count_launches(1);
  timing_end(kKernPstepGrad, stream);
  return err;
}

cudaError_t launch_adam(float* param, void* param_f16, const double* grad, float* exp_avg, float* exp_avg_sq,
                        uint64_t n, float lr, float beta1, float beta2, float eps, float bias1, float bias2,
                        int sm_count, cudaStream_t stream) {
  timing_begin(kKernAdam, stream);
  const uint64_t want = (n + 255) / 256, cap = (uint64_t)sm_count * 8;
  adam_kernel<<<(unsigned)(want < cap ? want : cap), 256, 0, stream>>>(param, reinterpret_cast<__half*>(param_f16), grad,
                                                                      exp_avg, exp_avg_sq, n, lr, beta1, beta2, eps,
                                                                      bias1, bias2);
  count_launches(1);
  timing_end(kKernAdam, stream);
  return cudaGetLastError();
}

}  // namespace pvt
