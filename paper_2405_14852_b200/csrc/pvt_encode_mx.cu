// Beam search for three or four additive codebooks (Appendix C / Appendix J: beam search, beam size 8; the
// residual form of the two-codebook kernel carried through more stages).
//
//   stage m (m = 1..M): each kept partial tuple (one empty tuple before stage 1) is extended by every codeword
//     of codebook m; the score of an extension is ||t - c^1 - ... - c^m||^2 with the residual carried in binary64
//     through the codebooks in order and the terms added in element order;
//   after stages 1..M-1 the `beam` smallest extensions under (score, tuple) are kept;
//   the result is the smallest member of the last stage's extensions and the previous tuple.
//
// One warp per target.  Codebooks sit in shared memory as binary32 (M * K * 32 bytes).  A stage makes two passes
// over fast estimates of all extensions: the first finds a threshold (the keep-th smallest of the lanes' minima),
// the second gives every extension within the estimates' error bound of it its binary64 score and keeps the
// lane's `beam` smallest in registers (sorted by insertion); the warp then extracts the overall `beam` smallest by
// repeated warp minimum over the lanes' heads.  For fp16 codebooks the estimates come from the tensor pipe: 16
// codewords are the rows [ c | c ] of an fp16 tile, the kept residuals its columns [ -hi(2^e r) | -lo(2^e r) ],
// the accumulator starts at 2^e ||c||^2 / 2 (mma.sync m16n8k16, fp32 accumulation): 16 instructions per pass over
// 256 codewords.  For binary32 codebooks, and for a stage with one or two kept residuals (the first), the estimate
// is sum_i (fl32(r_i) - c_i)^2 on the FP32 pipe.
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

constexpr int kMxCand = 256;              // capacity of a warp's candidate list
constexpr int kMxPadK = 256;              // codewords per codebook in the tensor-pipe image (padded)
constexpr float kMxPadHalfNorm = 3.0e38f;  // half norm of a padding codeword: never within any bound

// D = A (16 x 16, rows = codewords, each [ c | c ]) x B (16 x 8, columns = residuals, each [ -hi | -lo ]) + C,
// fp16 operands, fp32 accumulation.  A thread passes the words of rows lane/4 and lane/4 + 8 (the same word serves
// both halves of the depth) and the half norms of those two codewords as the start of the accumulator.
__device__ __forceinline__ void mma_cw16(float (&d)[4], uint32_t a_row, uint32_t a_row8, uint32_t b_hi, uint32_t b_lo,
                                         float c_row, float c_row8) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %4, %5}, {%6, %7}, "
      "{%8, %8, %9, %9};"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a_row), "r"(a_row8), "r"(b_hi), "r"(b_lo), "f"(c_row), "f"(c_row8));
}

// bytes of the tensor-pipe image of the codebooks: B fragments, half norms, largest norm per codebook
__host__ __device__ constexpr size_t mx_image_bytes(int M) {
  return (size_t)M * (kMxPadK / 8) * 32 * 4 + (size_t)M * kMxPadK * 4 + 16;
}

// bytes of everything the kernel derives from the codebooks (binary32 copy, and for fp16 codebooks the tensor-pipe
// image), in the byte order it has at the start of shared memory: a multiple of 16
__host__ __device__ constexpr size_t mx_staged_bytes(int M, uint32_t K, bool f16) {
  return (size_t)M * K * 32 + (f16 ? mx_image_bytes(M) : 0);
}

// Writes that image into the workspace, once per call (one block).
//   book   [M][K][8] binary32
//   fp16 codebooks only: A fragments, words [m][tile][lane][2] = halves (c[16 tile + lane/4 (+ 8)][2 (lane%4)], [.. + 1]);
//   ||c||^2/2 as [m][tile][lane/4][2]; max ||c||^2 per codebook (bit patterns)
template <int M, bool CB_F16>
__global__ void __launch_bounds__(kMxThreads) mx_image_kernel(const MxParams p, unsigned char* __restrict__ out) {
  const uint32_t K = p.K;
  float* book = reinterpret_cast<float*>(out);
  uint32_t* bfrag = reinterpret_cast<uint32_t*>(out + (size_t)M * K * 32);
  float* hnorm = reinterpret_cast<float*>(bfrag + M * (kMxPadK / 8) * 32);
  uint32_t* n2max_bits = reinterpret_cast<uint32_t*>(hnorm + M * kMxPadK);
  if (CB_F16) {
    for (uint32_t e = threadIdx.x; e < (uint32_t)M * kMxPadK; e += kMxThreads) {
      hnorm[e] = kMxPadHalfNorm;
#pragma unroll
      for (int qq = 0; qq < 4; ++qq) bfrag[4 * e + qq] = 0u;
    }
    if (threadIdx.x < 4) n2max_bits[threadIdx.x] = 0u;
    __syncthreads();
  }
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
    if (CB_F16) {
      const uint32_t m = row / K, kap = row % K;
      float n2 = 0.0f;
#pragma unroll
      for (int i = 0; i < 8; ++i) n2 = fmaf(c[i], c[i], n2);
      // 16 codewords per tile: codeword 16 mt + r sits in row r; a thread of the warp reads rows g and g + 8
      const uint32_t mt = kap >> 4, g = kap & 7u, upper = (kap >> 3) & 1u;
      hnorm[((m * (kMxPadK / 16) + mt) * 8 + g) * 2 + upper] = 0.5f * n2;
      atomicMax(&n2max_bits[m], __float_as_uint(n2));  // non-negative: bits order like values
#pragma unroll
      for (int qq = 0; qq < 4; ++qq) {
        const __half2 v = __floats2half2_rn(c[2 * qq], c[2 * qq + 1]);  // exact: the codebook is fp16
        bfrag[((m * (kMxPadK / 16) + mt) * 32 + 4 * g + qq) * 2 + upper] = *reinterpret_cast<const uint32_t*>(&v);
      }
    }
  }
}

constexpr uint32_t kMxMaxSpins = 1u << 22;  // polls after which the wait for the image gives up

template <int M, bool CB_F16>
__global__ void __launch_bounds__(kMxThreads, M == 3 ? 4 : 3) encode_mx_kernel(const MxParams p,
                                                                                const unsigned char* __restrict__ image) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const uint32_t K = p.K;
  const size_t staged = mx_staged_bytes(M, K, CB_F16);
  // the codebooks' image, fetched with one bulk copy (cp.async.bulk, completion on an mbarrier; no multicast)
  float* book = reinterpret_cast<float*>(smem_raw);                               // [M][K][8]
  uint32_t* bfrag = reinterpret_cast<uint32_t*>(smem_raw + (size_t)M * K * 32);
  float* hnorm = reinterpret_cast<float*>(bfrag + M * (kMxPadK / 8) * 32);
  uint32_t* n2max_bits = reinterpret_cast<uint32_t*>(hnorm + M * kMxPadK);
  // scratch behind it
  double* resid = reinterpret_cast<double*>(smem_raw + staged);                   // [warps][beam][8]
  float* resid_f = reinterpret_cast<float*>(resid + kMxWarps * kMxBeam * 8);      // the same, rounded to binary32
  // per warp: the extensions that pass the filter of a stage, (kept tuple << 8 | code), and their count
  uint16_t* cand = reinterpret_cast<uint16_t*>(resid_f + kMxWarps * kMxBeam * 8);
  uint32_t* cand_n = reinterpret_cast<uint32_t*>(cand + kMxWarps * kMxCand);
  // per warp: the kept partial tuples and the target
  uint32_t* kept_sm = cand_n + kMxWarps;
  float* t_sm = reinterpret_cast<float*>(kept_sm + kMxWarps * kMxBeam);
  uint64_t* img_bar = reinterpret_cast<uint64_t*>(t_sm + kMxWarps * 8);
  {
    const uint32_t b = (uint32_t)__cvta_generic_to_shared(img_bar);
    if (threadIdx.x == 0) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(b));
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b), "r"((uint32_t)staged) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                       (uint32_t)__cvta_generic_to_shared(smem_raw)),
                   "l"(image), "r"((uint32_t)staged), "r"(b)
                   : "memory");
    }
    __syncthreads();  // the barrier is initialised before anybody polls it
    uint32_t ok = 0;
    for (uint32_t spin = 0; spin < kMxMaxSpins && !ok; ++spin) {
      asm volatile(
          "{\n\t.reg .pred q;\n\t"
          "mbarrier.try_wait.parity.shared::cta.b64 q, [%1], 0;\n\t"
          "selp.u32 %0, 1, 0, q;\n\t}"
          : "=r"(ok)
          : "r"(b)
          : "memory");
      if (!ok && spin > 4096) __nanosleep(64);
    }
    if (!ok) atomicOr(p.status, PVT_DEV_WAIT_EXPIRED);
    if (!__syncthreads_and((int)ok)) return;  // the image has not landed: nobody reads it
  }

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // persistent: the resident warps share out the targets
#pragma unroll 1
  for (uint64_t n = (uint64_t)blockIdx.x * kMxWarps + warp; n < p.k; n += (uint64_t)gridDim.x * kMxWarps) {
  __syncwarp();  // the warp's scratch of the previous target is no longer read
  const uint32_t j = __ldg(p.idx + n);
  if (j >= p.G) {
    if (lane == 0) atomicOr(p.status, PVT_DEV_BAD_INDEX);
    continue;
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
  uint16_t* my_cand = cand + (size_t)warp * kMxCand;
  uint32_t* my_cand_n = cand_n + warp;
  uint32_t* my_kept = kept_sm + (size_t)warp * kMxBeam;
  float* my_t = t_sm + (size_t)warp * 8;
  const int beam = p.beam;

  // kept partial tuples: key = code_1 << 24 | code_2 << 16 | ... (lexicographic order of tuples = numeric order)
  // (they live in shared memory: every use picks one by a run-time index)
  int n_kept = 1;
  if (lane == 0) {
    my_kept[0] = 0u;
    *reinterpret_cast<float4*>(my_t) = make_float4(t[0], t[1], t[2], t[3]);
    *reinterpret_cast<float4*>(my_t + 4) = make_float4(t[4], t[5], t[6], t[7]);
  }
  double best_d = __longlong_as_double(kInfBits);
  uint32_t best_key = kNoKey;

#pragma unroll 1
  for (int m = 0; m < M; ++m) {
    // residuals of the kept tuples, carried in binary64 through the codebooks in order
    __syncwarp();
    for (int item = lane; item < n_kept * 8; item += 32) {
      const int b = item >> 3, i = item & 7;
      const uint32_t key = my_kept[b];
      double r = (double)my_t[i];
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

    double ld[kMxBeam];
    uint32_t lk[kMxBeam];
#pragma unroll
    for (int q = 0; q < kMxBeam; ++q) {
      ld[q] = __longlong_as_double(kInfBits);
      lk[q] = kNoKey;
    }
    // sorted insertion of an extension into this lane's list of `keep` entries: the new entry sinks to its place,
    // the last one drops
    auto insert = [&](double d, uint32_t key) {
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
    };
    // an extension that passed the filter goes on the warp's list (any order: the decision below does not depend
    // on it); a list that overflows is detected by its count
    if (lane == 0) *my_cand_n = 0u;
    __syncwarp();
    auto collect = [&](uint32_t b, uint32_t q) {
      const uint32_t pos = atomicAdd(my_cand_n, 1u);
      if (pos < (uint32_t)kMxCand) my_cand[pos] = (uint16_t)((b << 8) | q);
    };
    // binary64 score of extension (kept tuple b, codeword q of this stage's codebook) into this lane's list
    auto score_exact = [&](uint32_t b, uint32_t q, bool first) {
      const double* r = &my_resid[b * 8];
      const float* c = &book[((size_t)m * K + q) * 8];
      double d = 0.0;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const double ee = __dsub_rn(r[i], (double)c[i]);
        d = __dadd_rn(d, __dmul_rn(ee, ee));
      }
      const uint32_t key = my_kept[b] | (q << shift);
      if (first) {  // the list is still empty
        ld[0] = d;
        lk[0] = key;
      } else {
        insert(d, key);
      }
    };
    // theta: the keep-th smallest of the lanes' smallest estimates (one or two per lane, sorted) -- `keep` different
    // extensions have an estimate of at most theta, so the exact keep-th smallest score lies within the error bound
    // of it (a little looser than the keep-th smallest estimate overall, at a few instructions per extension instead
    // of a sorted insertion)
    auto kth_of_lane_minima = [&](uint32_t first, uint32_t second) {
      uint32_t theta_bits = 0x7f800000u;
      for (int round = 0; round < keep; ++round) {
        const uint32_t mv = __reduce_min_sync(0xffffffffu, first);
        theta_bits = mv;
        if (mv == 0x7f800000u) break;  // fewer than `keep` extensions on offer: everything survives
        const uint32_t owners = __ballot_sync(0xffffffffu, first == mv);
        if (lane == __ffs(owners) - 1) {  // equal minima in several lanes: one leaves per round
          first = second;
          second = 0x7f800000u;
        }
      }
      return theta_bits;
    };
    if (CB_F16 && n_kept >= 3) {  // with one or two kept residuals (the first stage) the FP32 pipe is cheaper
      // Estimates from the tensor pipe.  The kept residuals are the columns of B (column n = residual n, as
      // [ -hi(2^e r) | -lo(2^e r) ]), 16 codewords the rows of A.  A thread sees, per tile of 16 codewords, the
      // estimates of residuals 2 (lane % 4) and the next one against codewords 16 mt + lane / 4 and that + 8:
      //   est = ||r_f||^2 + 2 * 2^-e * D,   D = 2^e (||c||^2/2 - <r_f, c>)  up to rounding.
      // Error against the binary64 score d (R = largest residual norm, C = largest codeword norm, S = (R + C)^2):
      // rounding r to binary32 2^-23 sqrt(d) R; the halves 2^-21 R C, or 2^-24 2^-e sqrt(8) C where the low half is
      // subnormal; 17 accumulations of the products 2^-17.9 (R C + C^2/2); the norms 2^-20 C^2 + 2^-21 R^2:
      // below 2^-17 S + 2^-22 2^-e C in all.
      const uint32_t g8 = (uint32_t)lane >> 2, qd = (uint32_t)lane & 3u;
      const uint32_t nk = (uint32_t)n_kept;
      // the column this thread contributes to B: residual g8, elements 2 qd and 2 qd + 1
      float2 rv = make_float2(0.0f, 0.0f);
      if (g8 < nk) rv = *reinterpret_cast<const float2*>(&my_resid_f[g8 * 8 + 2 * qd]);
      // the two residuals whose estimates this thread receives, and their squared norms
      const uint32_t b0 = 2u * qd, b1 = 2u * qd + 1u;
      const bool valid0 = b0 < nk, valid1 = b1 < nk;
      auto sq_norm = [&](uint32_t b) {
        const float4 ra = *reinterpret_cast<const float4*>(&my_resid_f[b * 8]);
        const float4 rb = *reinterpret_cast<const float4*>(&my_resid_f[b * 8 + 4]);
        float rr = ra.x * ra.x;
        rr = fmaf(ra.y, ra.y, rr); rr = fmaf(ra.z, ra.z, rr); rr = fmaf(ra.w, ra.w, rr);
        rr = fmaf(rb.x, rb.x, rr); rr = fmaf(rb.y, rb.y, rr); rr = fmaf(rb.z, rb.z, rr); rr = fmaf(rb.w, rb.w, rr);
        return rr;
      };
      const float inf_f = __uint_as_float(0x7f800000u);
      const float rr0 = valid0 ? sq_norm(b0) : inf_f, rr1 = valid1 ? sq_norm(b1) : inf_f;  // inf: never within a bound
      const float rmax = fmaxf(fabsf(rv.x), fabsf(rv.y));
      const uint32_t rbits = __reduce_max_sync(0xffffffffu, __float_as_uint(rmax));
      const float r2max = __uint_as_float(
          __reduce_max_sync(0xffffffffu, __float_as_uint(fmaxf(valid0 ? rr0 : 0.0f, valid1 ? rr1 : 0.0f))));
      int e = 126 - (int)((rbits >> 23) & 0xffu);
      e = e > 15 ? 15 : (e < -100 ? -100 : e);
      const float sc = __uint_as_float((uint32_t)(e + 127) << 23), inv = __uint_as_float((uint32_t)(127 - e) << 23);
      uint32_t b_hi, b_lo;
      {
        const float x = -rv.x * sc, y = -rv.y * sc;  // exact
        const __half2 hi = __floats2half2_rn(x, y);
        const float2 back = __half22float2(hi);
        const __half2 lo = __floats2half2_rn(x - back.x, y - back.y);
        b_hi = *reinterpret_cast<const uint32_t*>(&hi);
        b_lo = *reinterpret_cast<const uint32_t*>(&lo);
      }
      const uint2* af = reinterpret_cast<const uint2*>(bfrag) + (size_t)m * (kMxPadK / 16) * 32 + lane;
      const float2* hn = reinterpret_cast<const float2*>(hnorm) + (size_t)m * (kMxPadK / 16) * 8 + g8;
      const float two_inv = 2.0f * inv;
      const uint32_t n_tiles = (K + 15u) >> 4;
      // pass 1: this lane's two smallest estimates
      float m0 = inf_f, m1 = inf_f;
#pragma unroll 4
      for (uint32_t mt = 0; mt < n_tiles; ++mt) {
        const uint2 a = af[32 * mt];
        const float2 hh = hn[8 * mt];
        float d[4];
        mma_cw16(d, a.x, a.y, b_hi, b_lo, hh.x * sc, hh.y * sc);
        const float e00 = fmaf(d[0], two_inv, rr0), e01 = fmaf(d[1], two_inv, rr1);
        const float e10 = fmaf(d[2], two_inv, rr0), e11 = fmaf(d[3], two_inv, rr1);
        // the two smallest of the four, then of those and (m0, m1)
        const float lo_a = fminf(e00, e01), hi_a = fmaxf(e00, e01), lo_b = fminf(e10, e11), hi_b = fmaxf(e10, e11);
        const float t0 = fminf(lo_a, lo_b), t1 = fminf(fmaxf(lo_a, lo_b), fminf(hi_a, hi_b));
        const float n0 = fminf(m0, t0);
        m1 = fminf(fmaxf(m0, t0), fminf(m1, t1));
        m0 = n0;
      }
      // an estimate can come out slightly negative; the order of the bit patterns needs non-negative values
      const uint32_t theta_bits =
          kth_of_lane_minima(__float_as_uint(fmaxf(m0, 0.0f)), __float_as_uint(fmaxf(m1, 0.0f)));
      const float theta = __uint_as_float(theta_bits);
      const float cmax = sqrtf(__uint_as_float(n2max_bits[m]));
      const float reach = sqrtf(r2max) + cmax;
      // twice the error bound, with a factor 2 to spare
      const float bound = theta_bits == 0x7f800000u
                              ? theta
                              : theta + 3.0517578e-5f /* 2^-15 */ * reach * reach + 9.5367432e-7f /* 2^-20 */ * inv * cmax + 1e-37f;
      // pass 2: the same estimates again (bit for bit); the few extensions within the bound go on the list
#pragma unroll 4
      for (uint32_t mt = 0; mt < n_tiles; ++mt) {
        const uint2 a = af[32 * mt];
        const float2 hh = hn[8 * mt];
        float d[4];
        mma_cw16(d, a.x, a.y, b_hi, b_lo, hh.x * sc, hh.y * sc);
        const float e00 = fmaf(d[0], two_inv, rr0), e01 = fmaf(d[1], two_inv, rr1);
        const float e10 = fmaf(d[2], two_inv, rr0), e11 = fmaf(d[3], two_inv, rr1);
        const uint32_t q = 16u * mt + g8;
        if (fminf(fminf(e00, e01), fminf(e10, e11)) <= bound) {
          if (valid0 && e00 <= bound && q < K) collect(b0, q);
          if (valid1 && e01 <= bound && q < K) collect(b1, q);
          if (valid0 && e10 <= bound && q + 8u < K) collect(b0, q + 8u);
          if (valid1 && e11 <= bound && q + 8u < K) collect(b1, q + 8u);
        }
      }
    } else {
      // Pass 1, binary32 and branch-free: the estimate d_fl = sum_i (fl32(r_i) - c_i)^2 of every extension.  With
      // R = the largest residual norm, |d_fl - d| <= 2^-22 sqrt(d) R + 2^-20 d: the residual is rounded to binary32
      // (2^-24 |r_i| per element, which matters when the codeword nearly cancels it), the differences, squares and
      // sums add relative roundings.
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
      // every member of the exact `keep` smallest has an estimate within the two error bounds of theta
      const uint32_t theta_bits = kth_of_lane_minima(est_min, 0x7f800000u);
      const float theta = __uint_as_float(theta_bits);
      const float bound = theta_bits == 0x7f800000u
                              ? theta
                              : theta + 4.0f * (2.3841858e-7f /* 2^-22 */ * sqrtf(theta * r2max) + 9.5367432e-7f /* 2^-20 */ * theta) +
                                    1e-37f;
      // Pass 2: the same estimates again (bit for bit); the few extensions within the bound go on the list
      for (int b = 0; b < n_kept; ++b) {
        const float4 ra = *reinterpret_cast<const float4*>(&my_resid_f[b * 8]);
        const float4 rb = *reinterpret_cast<const float4*>(&my_resid_f[b * 8 + 4]);
        for (uint32_t q = lane; q < K; q += 32)
          if (estimate(ra, rb, &book[((size_t)m * K + q) * 8]) <= bound) collect((uint32_t)b, q);
      }
    }

    // binary64 scores of the listed extensions, one per lane and round; a list that overflowed (many equal
    // codewords, or fewer extensions than `keep`) is replaced by all extensions
    __syncwarp();
    const uint32_t n_cand = *my_cand_n;
    {
      if (n_cand <= (uint32_t)kMxCand) {
        for (uint32_t i = lane; i < n_cand; i += 32) {
          const uint32_t e = my_cand[i];
          score_exact(e >> 8, e & 0xffu, i < 32u);
        }
      } else {
        for (uint32_t b = 0; b < (uint32_t)n_kept; ++b)
          for (uint32_t q = lane; q < K; q += 32) score_exact(b, q, false);
      }
    }

    // the warp's `keep` smallest under (score, tuple): repeated warp minimum over the lanes' current heads; with
    // at most one listed extension per lane the head is the lane's only entry
    __syncwarp();  // every lane has read the kept tuples it needed: they are replaced now
    int n_new = 0;
    const bool single = n_cand <= 32u;
    int head = 0;
    for (int round = 0; round < keep; ++round) {
      double hd = ld[0];
      uint32_t hk = lk[0];
      if (!single) {
#pragma unroll
        for (int x = 1; x < kMxBeam; ++x)
          if (x == head) {
            hd = ld[x];
            hk = lk[x];
          }
        if (head >= kMxBeam) {
          hd = __longlong_as_double(kInfBits);
          hk = kNoKey;
        }
      }
      const uint64_t bits = (uint64_t)__double_as_longlong(hd);
      const uint32_t hi = (uint32_t)(bits >> 32), lo = (uint32_t)bits;
      const uint32_t mhi = __reduce_min_sync(0xffffffffu, hi);
      const uint32_t mlo = __reduce_min_sync(0xffffffffu, hi == mhi ? lo : 0xffffffffu);
      const uint32_t mk = __reduce_min_sync(0xffffffffu, (hi == mhi && lo == mlo) ? hk : kNoKey);
      if (mhi == 0x7ff00000u && mlo == 0u) break;  // fewer candidates than `keep` (warp-uniform)
      if (hi == mhi && lo == mlo && hk == mk) {  // keys are unique: exactly one lane pops
        if (single) {
          ld[0] = __longlong_as_double(kInfBits);
          lk[0] = kNoKey;
        } else {
          ++head;
        }
      }
      if (m == M - 1) {
        best_d = __longlong_as_double((long long)(((uint64_t)mhi << 32) | mlo));
        best_key = mk;
      } else {
        if (lane == 0) my_kept[n_new] = mk;
        ++n_new;
      }
    }
    if (m < M - 1) n_kept = n_new;
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
  }  // targets of this warp
}

template <int M, bool CB_F16>
cudaError_t launch_m(const MxParams& p, unsigned char* image, int sm_count, cudaStream_t stream) {
  const size_t smem = mx_staged_bytes(M, p.K, CB_F16) +
                      (size_t)kMxWarps * kMxBeam * 8 * (sizeof(double) + sizeof(float)) +
                      (size_t)kMxWarps * (kMxCand * sizeof(uint16_t) + sizeof(uint32_t) + kMxBeam * 4 + 8 * 4) + 16;
  cudaError_t e = cudaFuncSetAttribute(encode_mx_kernel<M, CB_F16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  mx_image_kernel<M, CB_F16><<<1, kMxThreads, 0, stream>>>(p, image);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  int per_sm = 0;
  if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, encode_mx_kernel<M, CB_F16>, kMxThreads, smem)) !=
      cudaSuccess)
    return e;
  const uint64_t needed = (p.k + kMxWarps - 1) / kMxWarps;
  const uint64_t resident = (uint64_t)sm_count * (uint64_t)(per_sm > 0 ? per_sm : 1);
  encode_mx_kernel<M, CB_F16><<<(unsigned)(needed < resident ? needed : resident), kMxThreads, smem, stream>>>(p, image);
  count_launches(2);
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
  unsigned char* image = static_cast<unsigned char*>(ws) + kWsHeaderBytes;
  const int sms = device_sm_count();
  if (L.num_codebooks == 3)
    e = f16 ? launch_m<3, true>(p, image, sms, stream) : launch_m<3, false>(p, image, sms, stream);
  else
    e = f16 ? launch_m<4, true>(p, image, sms, stream) : launch_m<4, false>(p, image, sms, stream);
  timing_end(kKernEncodeMain, stream);
  return e;
}

}  // namespace pvt
