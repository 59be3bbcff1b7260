// Beam search for three or four additive codebooks (Appendix C / Appendix J: beam search, beam size 8; the
// residual form of the two-codebook kernel carried through more stages).  First version: every candidate is
// scored directly in binary64, exactly as the decision is defined, so there is no fast filter and no rescoring:
//
//   stage m (m = 1..M): each kept partial tuple (one empty tuple before stage 1) is extended by every codeword
//     of codebook m; the score of an extension is ||t - c^1 - ... - c^m||^2 with the residual carried in binary64
//     through the codebooks in order and the terms added in element order;
//   after stages 1..M-1 the `beam` smallest extensions under (score, tuple) are kept;
//   the result is the smallest member of the last stage's extensions and the previous tuple.
//
// One warp per target.  Codebooks sit in shared memory as binary32 (M * K * 32 bytes).  Per stage a lane scores
// the candidates lane, lane+32, ... and keeps its own `beam` smallest in registers (sorted by insertion); the
// warp then extracts the overall `beam` smallest by repeated warp minimum over the lanes' heads.
// Cost per target: (1 + (M-1) * beam) * K candidates of 24 binary64 operations.
#include <cuda_fp16.h>

#include "pvt_internal.h"

namespace pvt {
namespace {

constexpr int kMxThreads = 256;
constexpr int kMxWarps = kMxThreads / 32;
constexpr int kMxBeam = 8;
constexpr uint32_t kNoKey = 0xffffffffu;
constexpr long long kInfBits = 0x7ff0000000000000ll;

struct MxParams {
  const float* W;
  const float* g;
  const float* scale;
  const void* books;
  uint8_t* codes;
  const uint32_t* idx;
  uint64_t k, G;
  uint32_t gpr, K;
  int beam;
  float eta;
  float* err_out;
  uint32_t* status;
};

// (score, key) lexicographic; scores are >= 0 or +inf, never NaN for finite inputs
__device__ __forceinline__ bool less_than(double da, uint32_t ka, double db, uint32_t kb) {
  return da < db || (da == db && ka < kb);
}

template <int M, bool CB_F16>
__global__ void __launch_bounds__(kMxThreads) encode_mx_kernel(const MxParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* book = reinterpret_cast<float*>(smem_raw);                               // [M][K][8]
  double* resid = reinterpret_cast<double*>(smem_raw + (size_t)M * p.K * 32);     // [warps][beam][8]
  float* resid_f = reinterpret_cast<float*>(resid + kMxWarps * kMxBeam * 8);      // the same, rounded to binary32
  const uint32_t K = p.K;
  for (uint32_t row = threadIdx.x; row < M * K; row += kMxThreads) {
    float c[8];
    if (CB_F16) {
      const uint4 raw = __ldg(reinterpret_cast<const uint4*>(p.books) + row);
      const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
        c[2 * i] = f.x;
        c[2 * i + 1] = f.y;
      }
    } else {
      const float4* src = reinterpret_cast<const float4*>(p.books) + 2 * (size_t)row;
      const float4 lo = __ldg(src), hi = __ldg(src + 1);
      c[0] = lo.x, c[1] = lo.y, c[2] = lo.z, c[3] = lo.w, c[4] = hi.x, c[5] = hi.y, c[6] = hi.z, c[7] = hi.w;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) book[(size_t)row * 8 + i] = c[i];
  }
  __syncthreads();

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint64_t n = (uint64_t)blockIdx.x * kMxWarps + warp;
  if (n >= p.k) return;
  const uint32_t j = __ldg(p.idx + n);
  if (j >= p.G) {
    if (lane == 0) atomicOr(p.status, PVT_DEV_BAD_INDEX);
    return;
  }
  // target (Eq. 8 in the scaled space): one fma and one division per element, binary32
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
  double* my_resid = resid + (size_t)warp * kMxBeam * 8;
  float* my_resid_f = resid_f + (size_t)warp * kMxBeam * 8;
  const int beam = p.beam;

  // kept partial tuples: key = code_1 << 24 | code_2 << 16 | ... (lexicographic order of tuples = numeric order)
  uint32_t kept_key[kMxBeam];
  int n_kept = 1;
  kept_key[0] = 0;
#pragma unroll
  for (int b = 1; b < kMxBeam; ++b) kept_key[b] = 0;
  double best_d = __longlong_as_double(kInfBits);
  uint32_t best_key = kNoKey;

#pragma unroll 1
  for (int m = 0; m < M; ++m) {
    // residuals of the kept tuples, carried in binary64 through the codebooks in order
    __syncwarp();
    for (int item = lane; item < n_kept * 8; item += 32) {
      const int b = item >> 3, i = item & 7;
      uint32_t key = kept_key[0];
#pragma unroll
      for (int q = 1; q < kMxBeam; ++q)
        if (q == b) key = kept_key[q];
      double r = (double)t[0];
#pragma unroll
      for (int q = 1; q < 8; ++q)
        if (q == i) r = (double)t[q];
      for (int q = 0; q < m; ++q) {
        const uint32_t code = (key >> (24 - 8 * q)) & 0xffu;
        r = __dsub_rn(r, (double)book[((size_t)q * K + code) * 8 + i]);
      }
      my_resid[b * 8 + i] = r;
      my_resid_f[b * 8 + i] = (float)r;
    }
    __syncwarp();

    const int keep = (m == M - 1) ? 1 : beam;
    const int shift = 24 - 8 * m;

    // Pass 1, binary32 and branch-free: the estimate d_fl = sum_i (fl32(r_i) - c_i)^2 of every extension; each lane
    // keeps its smallest estimate, the warp derives a threshold theta from the 32 minima.  With R = the largest residual norm, |d_fl - d| <= 2^-22 sqrt(d) R + 2^-20 d: the residual is
    // rounded to binary32 (2^-24 |r_i| per element, which matters when the codeword nearly cancels it), the
    // differences, squares and sums add relative roundings.
    float r2max = 0.0f;
    if (lane < n_kept) {
#pragma unroll
      for (int i = 0; i < 8; ++i) r2max = fmaf(my_resid_f[lane * 8 + i], my_resid_f[lane * 8 + i], r2max);
    }
    r2max = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(r2max)));  // non-negative: bits order like values
    auto estimate = [&](const float4& ra, const float4& rb, const float* c) {
      const float4 ca = *reinterpret_cast<const float4*>(c), cb = *reinterpret_cast<const float4*>(c + 4);
      float e, dfl;
      e = ra.x - ca.x; dfl = e * e;
      e = ra.y - ca.y; dfl = fmaf(e, e, dfl);
      e = ra.z - ca.z; dfl = fmaf(e, e, dfl);
      e = ra.w - ca.w; dfl = fmaf(e, e, dfl);
      e = rb.x - cb.x; dfl = fmaf(e, e, dfl);
      e = rb.y - cb.y; dfl = fmaf(e, e, dfl);
      e = rb.z - cb.z; dfl = fmaf(e, e, dfl);
      e = rb.w - cb.w; dfl = fmaf(e, e, dfl);
      return dfl;
    };
    uint32_t est_min = 0x7f800000u;  // this lane's smallest estimate (non-negative: bits order like values)
    for (int b = 0; b < n_kept; ++b) {
      const float4 ra = *reinterpret_cast<const float4*>(&my_resid_f[b * 8]);
      const float4 rb = *reinterpret_cast<const float4*>(&my_resid_f[b * 8 + 4]);
      for (uint32_t q = lane; q < K; q += 32)
        est_min = min(est_min, __float_as_uint(estimate(ra, rb, &book[((size_t)m * K + q) * 8])));
    }
    // theta: the keep-th smallest of the 32 lane minima -- `keep` different extensions have an estimate of at
    // most theta, so the exact keep-th smallest score lies within the error bound of it (a little looser than
    // the keep-th smallest estimate overall, at one instruction per extension instead of a sorted insertion)
    uint32_t theta_bits = 0x7f800000u;
    {
      uint32_t hv = est_min;
      for (int round = 0; round < keep; ++round) {
        const uint32_t mv = __reduce_min_sync(0xffffffffu, hv);
        if (mv == 0x7f800000u) {  // fewer than `keep` lanes have an extension: everything survives
          theta_bits = mv;
          break;
        }
        theta_bits = mv;
        const uint32_t owners = __ballot_sync(0xffffffffu, hv == mv);
        if (lane == __ffs(owners) - 1) hv = 0x7f800000u;  // equal minima in several lanes: one leaves per round
      }
    }
    // every member of the exact `keep` smallest has an estimate within the two error bounds of theta
    const float theta = __uint_as_float(theta_bits);
    const float bound = theta_bits == 0x7f800000u
                            ? theta
                            : theta + 4.0f * (2.3841858e-7f /* 2^-22 */ * sqrtf(theta * r2max) + 9.5367432e-7f /* 2^-20 */ * theta) +
                                  1e-37f;

    // Pass 2: the same estimates again (bit for bit); the few extensions within the bound are scored in binary64
    // and kept in this lane's sorted list
    double ld[kMxBeam];
    uint32_t lk[kMxBeam];
#pragma unroll
    for (int q = 0; q < kMxBeam; ++q) {
      ld[q] = __longlong_as_double(kInfBits);
      lk[q] = kNoKey;
    }
    for (int b = 0; b < n_kept; ++b) {
      const float4 ra = *reinterpret_cast<const float4*>(&my_resid_f[b * 8]);
      const float4 rb = *reinterpret_cast<const float4*>(&my_resid_f[b * 8 + 4]);
      uint32_t kb = kept_key[0];
#pragma unroll
      for (int x = 1; x < kMxBeam; ++x)
        if (x == b) kb = kept_key[x];
      const double* r = &my_resid[b * 8];
      for (uint32_t q = lane; q < K; q += 32) {
        const float* c = &book[((size_t)m * K + q) * 8];
        if (!(estimate(ra, rb, c) <= bound)) continue;
        double d = 0.0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const double ee = __dsub_rn(r[i], (double)c[i]);
          d = __dadd_rn(d, __dmul_rn(ee, ee));
        }
        uint32_t key = kb | (q << shift);
        // insertion into the sorted list of `keep` entries: the new entry sinks to its place, the last one drops
#pragma unroll
        for (int x = 0; x < kMxBeam; ++x) {
          if (x < keep && less_than(d, key, ld[x], lk[x])) {
            const double td = ld[x];
            const uint32_t tk = lk[x];
            ld[x] = d;
            lk[x] = key;
            d = td;
            key = tk;
          }
        }
      }
    }

    // the warp's `keep` smallest: repeated minimum over the lanes' current heads
    int head = 0;
    uint32_t new_key[kMxBeam];
#pragma unroll
    for (int x = 0; x < kMxBeam; ++x) new_key[x] = 0;
    int n_new = 0;
    for (int round = 0; round < keep; ++round) {
      double hd = __longlong_as_double(kInfBits);
      uint32_t hk = kNoKey;
#pragma unroll
      for (int x = 0; x < kMxBeam; ++x)
        if (x == head) {
          hd = ld[x];
          hk = lk[x];
        }
      const uint64_t bits = (uint64_t)__double_as_longlong(hd);
      const uint32_t hi = (uint32_t)(bits >> 32), lo = (uint32_t)bits;
      const uint32_t mhi = __reduce_min_sync(0xffffffffu, hi);
      const uint32_t mlo = __reduce_min_sync(0xffffffffu, hi == mhi ? lo : 0xffffffffu);
      const uint32_t mk = __reduce_min_sync(0xffffffffu, (hi == mhi && lo == mlo) ? hk : kNoKey);
      if (mhi == 0x7ff00000u && mlo == 0u) break;  // fewer candidates than `keep` (warp-uniform)
      if (hi == mhi && lo == mlo && hk == mk) ++head;  // keys are unique: exactly one lane pops
      if (m == M - 1) {
        best_d = __longlong_as_double((long long)(((uint64_t)mhi << 32) | mlo));
        best_key = mk;
      } else {
#pragma unroll
        for (int x = 0; x < kMxBeam; ++x)
          if (x == n_new) new_key[x] = mk;
        ++n_new;
      }
    }
    if (m < M - 1) {
#pragma unroll
      for (int x = 0; x < kMxBeam; ++x) kept_key[x] = new_key[x];
      n_kept = n_new;
    }
  }

  // the previous tuple joins the pool (Lemma 3.3: the step never raises the error)
  {
    const uint8_t* pc = p.codes + (size_t)j * M;
    uint32_t pkey = 0;
    bool ok = true;
#pragma unroll
    for (int q = 0; q < M; ++q) {
      const uint32_t c = pc[q];
      ok &= c < K;
      pkey |= c << (24 - 8 * q);
    }
    if (!ok) {
      if (lane == 0) atomicOr(p.status, PVT_DEV_BAD_CODE);
    } else {
      double d = 0.0;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        double r = (double)t[i];
#pragma unroll
        for (int q = 0; q < M - 1; ++q)
          r = __dsub_rn(r, (double)book[((size_t)q * K + ((pkey >> (24 - 8 * q)) & 0xffu)) * 8 + i]);
        const double e =
            __dsub_rn(r, (double)book[((size_t)(M - 1) * K + ((pkey >> (24 - 8 * (M - 1))) & 0xffu)) * 8 + i]);
        d = __dadd_rn(d, __dmul_rn(e, e));
      }
      if (less_than(d, pkey, best_d, best_key)) {
        best_d = d;
        best_key = pkey;
      }
    }
  }
  if (lane == 0) {
    if (!(best_d < __longlong_as_double(kInfBits))) {
      atomicOr(p.status, PVT_DEV_INTERNAL);
    } else {
      uint8_t* out = p.codes + (size_t)j * M;
#pragma unroll
      for (int q = 0; q < M; ++q) out[q] = (uint8_t)((best_key >> (24 - 8 * q)) & 0xffu);
      if (p.err_out) p.err_out[n] = (float)best_d;
    }
  }
}

template <int M, bool CB_F16>
cudaError_t launch_m(const MxParams& p, cudaStream_t stream) {
  const size_t smem = (size_t)M * p.K * 32 + (size_t)kMxWarps * kMxBeam * 8 * (sizeof(double) + sizeof(float));
  cudaError_t e = cudaFuncSetAttribute(encode_mx_kernel<M, CB_F16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  const unsigned blocks = (unsigned)((p.k + kMxWarps - 1) / kMxWarps);
  encode_mx_kernel<M, CB_F16><<<blocks, kMxThreads, smem, stream>>>(p);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_encode_mx(const pvt_layer& L, uint64_t G, const uint32_t* idx, uint64_t k, float* err_out,
                             void* ws, cudaStream_t stream) {
  MxParams p;
  p.W = L.W;
  p.g = L.g;
  p.scale = L.scale;
  p.books = L.codebooks;
  p.codes = static_cast<uint8_t*>(L.codes);
  p.idx = idx;
  p.k = k;
  p.G = G;
  p.gpr = (uint32_t)(L.cols / kGroupDim);
  p.K = (uint32_t)L.codebook_size;
  p.beam = L.beam;
  p.eta = L.eta;
  p.err_out = err_out;
  p.status = static_cast<uint32_t*>(ws);
  const bool f16 = L.codebook_dtype == PVT_F16;
  timing_begin(kKernEncodeMain, stream);
  cudaError_t e;
  if (L.num_codebooks == 3)
    e = f16 ? launch_m<3, true>(p, stream) : launch_m<3, false>(p, stream);
  else
    e = f16 ? launch_m<4, true>(p, stream) : launch_m<4, false>(p, stream);
  timing_end(kKernEncodeMain, stream);
  return e;
}

}  // namespace pvt
