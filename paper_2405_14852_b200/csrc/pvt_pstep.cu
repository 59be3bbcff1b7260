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

template <bool CB_F16>
__device__ __forceinline__ float4 half_codeword(const void* book, uint32_t code, uint32_t half) {
  if (CB_F16) {
    const uint2 raw = __ldg(reinterpret_cast<const uint2*>(book) + 2 * (size_t)code + half);
    const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
    const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
    return make_float4(lo.x, lo.y, hi.x, hi.y);
  } else {
    return __ldg(reinterpret_cast<const float4*>(book) + 2 * (size_t)code + half);
  }
}

__device__ __forceinline__ void red_add_f64(double* p, double v) {
  asm volatile("red.global.add.f64 [%0], %1;" ::"l"(p), "d"(v) : "memory");
}

template <int M, bool CB_F16, bool CODE_U16, bool SMEM_ACC>
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
  const uint64_t H = 2 * G;
  const float4* g4 = reinterpret_cast<const float4*>(g);
  const int lane = threadIdx.x & 31;
  for (uint64_t h0 = (uint64_t)blockIdx.x * kPsThreads; h0 < H; h0 += (uint64_t)gridDim.x * kPsThreads) {
    const uint64_t h = h0 + threadIdx.x;
    const bool valid = h < H;
    const uint32_t j = (uint32_t)(h >> 1), half = (uint32_t)h & 1u;
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
        b[0] = __ldg(reinterpret_cast<const uint8_t*>(codes) + j);
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
          const size_t at = ((size_t)m * K + b[m]) * 8 + half * 4;
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
          float4 v = half_codeword<CB_F16>(codebooks, b[0], half);
          if (M == 2) {
            const float4 v2 = half_codeword<CB_F16>(codebooks, K + b[M - 1], half);
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

template <int M, bool CB_F16, bool CODE_U16>
cudaError_t launch_grad(const pvt_layer& L, uint64_t G, double* grad_books, double* grad_scale, uint32_t* status,
                        int sm_count, cudaStream_t stream) {
  const uint32_t gpr = (uint32_t)(L.cols / kGroupDim), K = (uint32_t)L.codebook_size;
  const bool smem_acc = (uint32_t)M * K <= (uint32_t)kPsSmemCodewords;
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
                                    sizeof(double) * (size_t)L.num_codebooks * (size_t)L.codebook_size * kGroupDim, stream);
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
  } else {
    if (f16)
      err = u16 ? launch_grad<2, true, true>(L, G, grad_books, grad_scale, status, sm_count, stream)
                : launch_grad<2, true, false>(L, G, grad_books, grad_scale, status, sm_count, stream);
    else
      err = u16 ? launch_grad<2, false, true>(L, G, grad_books, grad_scale, status, sm_count, stream)
                : launch_grad<2, false, false>(L, G, grad_books, grad_scale, status, sm_count, stream);
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
