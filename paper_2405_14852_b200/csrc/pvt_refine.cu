// Local search over single-code changes (Appendix D) for the groups of a subspace, started from the codes
// that are stored -- typically right after pvt_vstep_encode, whose beam search is a heuristic for two
// codebooks.  A move replaces one code of the group's tuple by the value that lowers ||t - sum_m C_m[b_m]||^2
// most (the neighbour that is smallest under (error, tuple)), and is taken only if the error strictly drops.
//
// One warp per target, one to four codebooks.  Every error is the binary64 sum the final decision of the search kernels uses
// (residual through the codebooks in order, terms added in element order), so the moves are decided on exact
// values and the error can only fall.  All M*K neighbours are evaluated per move: M*K*8 binary64 multiply-adds
// per target and move, a few moves per target.
#include <cuda_fp16.h>

#include "pvt_internal.h"

namespace pvt {
namespace {

constexpr int kRfThreads = 256;
constexpr int kRfSmemCodewords = 512;  // M*K up to this many codewords are staged in shared memory as binary32

struct RefineParams {
  const float* W;
  const float* g;
  const float* scale;
  const void* books;
  void* codes;
  const uint32_t* idx;
  uint64_t k, G;
  uint32_t gpr, K;
  float eta;
  int max_moves;
  float* err_out;
  uint32_t* moves_out;
  uint32_t* status;
};

template <bool CB_F16>
__device__ __forceinline__ void global_codeword(const void* books, uint32_t row, float c[8]) {
  if (CB_F16) {
    const uint4 raw = __ldg(reinterpret_cast<const uint4*>(books) + row);
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
      c[2 * i] = f.x;
      c[2 * i + 1] = f.y;
    }
  } else {
    const float4* src = reinterpret_cast<const float4*>(books) + 2 * (size_t)row;
    const float4 lo = __ldg(src), hi = __ldg(src + 1);
    c[0] = lo.x, c[1] = lo.y, c[2] = lo.z, c[3] = lo.w, c[4] = hi.x, c[5] = hi.y, c[6] = hi.z, c[7] = hi.w;
  }
}

// ||t - c_1 - ... - c_M||^2 with the residual carried in binary64 through the codebooks in order and the terms
// added in element order; cw[m] = the codeword of codebook m
template <int M>
__device__ __forceinline__ double tuple_error(const float t[8], const float (*cw)[8]) {
  double d = 0.0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    double e = (double)t[i];
#pragma unroll
    for (int m = 0; m < M; ++m) e = __dsub_rn(e, (double)cw[m][i]);
    d = __dadd_rn(d, __dmul_rn(e, e));
  }
  return d;
}

template <int M, bool CB_F16, bool CODE_U16, bool STAGED>
__global__ void __launch_bounds__(kRfThreads) refine_kernel(const RefineParams p) {
  __shared__ __align__(16) float sh_book[STAGED ? kRfSmemCodewords * 8 : 8];
  const uint32_t K = p.K;
  if (STAGED) {
    for (uint32_t row = threadIdx.x; row < M * K; row += kRfThreads) {
      float c[8];
      global_codeword<CB_F16>(p.books, row, c);
#pragma unroll
      for (int i = 0; i < 8; ++i) sh_book[row * 8 + i] = c[i];
    }
    __syncthreads();
  }
  auto codeword = [&](uint32_t row, float c[8]) {
    if (STAGED) {
      const float4 lo = *reinterpret_cast<const float4*>(&sh_book[row * 8]);
      const float4 hi = *reinterpret_cast<const float4*>(&sh_book[row * 8 + 4]);
      c[0] = lo.x, c[1] = lo.y, c[2] = lo.z, c[3] = lo.w, c[4] = hi.x, c[5] = hi.y, c[6] = hi.z, c[7] = hi.w;
    } else {
      global_codeword<CB_F16>(p.books, row, c);
    }
  };
  const int lane = threadIdx.x & 31;
  const uint64_t n = (uint64_t)blockIdx.x * (kRfThreads / 32) + (threadIdx.x >> 5);
  if (n >= p.k) return;
  const uint32_t j = __ldg(p.idx + n);
  if (j >= p.G) {
    if (lane == 0 && p.status) atomicOr(p.status, PVT_DEV_BAD_INDEX);
    return;
  }
  // target of the search (Eq. 8 in the scaled space): one fma and one division per element, binary32
  float t[8];
  {
    const float4* W4 = reinterpret_cast<const float4*>(p.W) + 2 * (size_t)j;
    const float4* g4 = reinterpret_cast<const float4*>(p.g) + 2 * (size_t)j;
    const float4 w0 = __ldg(W4), w1 = __ldg(W4 + 1), g0 = __ldg(g4), g1 = __ldg(g4 + 1);
    const float s = __ldg(p.scale + j / p.gpr), ne = -p.eta;
    const float w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
    const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) t[i] = __fdiv_rn(__fmaf_rn(ne, gg[i], w[i]), s);
  }
  uint32_t b[M];
  bool ok = true;
  if (M == 1) {
    b[0] = CODE_U16 ? reinterpret_cast<const uint16_t*>(p.codes)[j] : reinterpret_cast<const uint8_t*>(p.codes)[j];
  } else {
    const uint8_t* c = reinterpret_cast<const uint8_t*>(p.codes) + (size_t)j * M;
#pragma unroll
    for (int m = 0; m < M; ++m) b[m] = c[m];
  }
#pragma unroll
  for (int m = 0; m < M; ++m) ok = ok && b[m] < K;
  if (!ok) {
    if (lane == 0 && p.status) atomicOr(p.status, PVT_DEV_BAD_CODE);
    return;
  }
  float cw[M][8];
#pragma unroll
  for (int m = 0; m < M; ++m) codeword((uint32_t)m * K + b[m], cw[m]);
  double d_cur = tuple_error<M>(t, cw);
  uint32_t moves = 0;
  while (moves < (uint32_t)p.max_moves) {
    // best neighbour of this lane under (error, tuple); a neighbour is named by (codebook changed, new code)
    double ld = __longlong_as_double(0x7ff0000000000000ll);
    uint32_t lm = 0, lq = 0;
    bool lhave = false;
    auto tuple_less = [&](uint32_t m1, uint32_t q1, uint32_t m2, uint32_t q2) {
      // lexicographic order of the two neighbours' tuples (both differ from the current tuple in one place)
#pragma unroll
      for (int m = 0; m < M; ++m) {
        const uint32_t x = (uint32_t)m == m1 ? q1 : b[m], y = (uint32_t)m == m2 ? q2 : b[m];
        if (x != y) return x < y;
      }
      return false;
    };
#pragma unroll
    for (int m = 0; m < M; ++m) {
      float keep[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) keep[i] = cw[m][i];
      for (uint32_t q = lane; q < K; q += 32) {
        if (q == b[m]) continue;
        codeword((uint32_t)m * K + q, cw[m]);
        const double d = tuple_error<M>(t, cw);
        if (!lhave || d < ld || (d == ld && tuple_less((uint32_t)m, q, lm, lq))) {
          ld = d;
          lm = (uint32_t)m;
          lq = q;
          lhave = true;
        }
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) cw[m][i] = keep[i];
    }
    // warp-wide minimum of (error, tuple); errors are >= 0, so their bits order like u64
    const uint64_t bits = (uint64_t)__double_as_longlong(ld);
    const uint32_t hi = (uint32_t)(bits >> 32), lo = (uint32_t)bits;
    const uint32_t mhi = __reduce_min_sync(0xffffffffu, hi);
    const uint32_t mlo = __reduce_min_sync(0xffffffffu, hi == mhi ? lo : 0xffffffffu);
    const bool tied = lhave && hi == mhi && lo == mlo;
    // among the lanes that hold the minimum error: the smallest tuple, codebook by codebook
    uint32_t alive_mask = __ballot_sync(0xffffffffu, tied);
    if (alive_mask == 0 || !(__longlong_as_double((long long)(((uint64_t)mhi << 32) | mlo)) < d_cur)) break;
    bool mine = tied;
#pragma unroll
    for (int m = 0; m < M; ++m) {
      const uint32_t x = mine ? ((uint32_t)m == lm ? lq : b[m]) : 0xffffffffu;
      const uint32_t mx = __reduce_min_sync(0xffffffffu, x);
      mine = mine && x == mx;
    }
    const int winner = __ffs(__ballot_sync(0xffffffffu, mine)) - 1;  // exactly one lane (tuples are distinct)
    const uint32_t wm = __shfl_sync(0xffffffffu, lm, winner), wq = __shfl_sync(0xffffffffu, lq, winner);
#pragma unroll
    for (int m = 0; m < M; ++m)
      if ((uint32_t)m == wm) {
        b[m] = wq;
        codeword((uint32_t)m * K + wq, cw[m]);
      }
    d_cur = __longlong_as_double((long long)(((uint64_t)mhi << 32) | mlo));
    ++moves;
  }
  if (lane == 0) {
    if (moves) {
      if (M == 1) {
        if (CODE_U16)
          reinterpret_cast<uint16_t*>(p.codes)[j] = (uint16_t)b[0];
        else
          reinterpret_cast<uint8_t*>(p.codes)[j] = (uint8_t)b[0];
      } else {
        uint8_t* c = reinterpret_cast<uint8_t*>(p.codes) + (size_t)j * M;
#pragma unroll
        for (int m = 0; m < M; ++m) c[m] = (uint8_t)b[m];
      }
    }
    if (p.err_out) p.err_out[n] = (float)d_cur;
    if (p.moves_out) p.moves_out[n] = moves;
  }
}

template <int M, bool CB_F16, bool CODE_U16>
cudaError_t launch_staged(const RefineParams& p, cudaStream_t stream) {
  const unsigned blocks = (unsigned)((p.k + kRfThreads / 32 - 1) / (kRfThreads / 32));
  if ((uint64_t)M * p.K <= (uint64_t)kRfSmemCodewords)
    refine_kernel<M, CB_F16, CODE_U16, true><<<blocks, kRfThreads, 0, stream>>>(p);
  else
    refine_kernel<M, CB_F16, CODE_U16, false><<<blocks, kRfThreads, 0, stream>>>(p);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_refine(const pvt_layer& L, uint64_t G, const uint32_t* idx, uint64_t k, int max_moves,
                          float* err_out, uint32_t* moves_out, uint32_t* status, cudaStream_t stream) {
  RefineParams p;
  p.W = L.W;
  p.g = L.g;
  p.scale = L.scale;
  p.books = L.codebooks;
  p.codes = L.codes;
  p.idx = idx;
  p.k = k;
  p.G = G;
  p.gpr = (uint32_t)(L.cols / kGroupDim);
  p.K = (uint32_t)L.codebook_size;
  p.eta = L.eta;
  p.max_moves = max_moves;
  p.err_out = err_out;
  p.moves_out = moves_out;
  p.status = status;
  const bool f16 = L.codebook_dtype == PVT_F16, u16 = L.code_dtype == PVT_U16;
  timing_begin(kKernRefine, stream);
  cudaError_t e;
  if (L.num_codebooks == 2)
    e = f16 ? launch_staged<2, true, false>(p, stream) : launch_staged<2, false, false>(p, stream);
  else if (L.num_codebooks == 3)
    e = f16 ? launch_staged<3, true, false>(p, stream) : launch_staged<3, false, false>(p, stream);
  else if (L.num_codebooks == 4)
    e = f16 ? launch_staged<4, true, false>(p, stream) : launch_staged<4, false, false>(p, stream);
  else if (f16)
    e = u16 ? launch_staged<1, true, true>(p, stream) : launch_staged<1, true, false>(p, stream);
  else
    e = u16 ? launch_staged<1, false, true>(p, stream) : launch_staged<1, false, false>(p, stream);
  timing_end(kKernRefine, stream);
  return e;
}

}  // namespace pvt
