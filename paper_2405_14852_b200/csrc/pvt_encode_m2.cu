// Greedy residual beam search of the V step for two additive codebooks
// (Appendix C: the code combination is found by beam search; Appendix J:
// two 8-bit codebooks, group size 8, beam size 8, target = gradient-updated
// dequantised weight; Eq. 8 for the target; Lemma 3.3 for keeping the previous
// pair in the pool).
//
// A warp handles four targets at a time; both codebooks live in shared memory;
// three CTAs (24 warps) share an SM.
//   stage 1 (per target, the whole warp): lane l owns codewords l, l+32, ..., l+224
//            of codebook 1: score1 = ||c1||^2/2 - <t, c1> for 256 codewords (8 per
//            lane, packed f32x2); the `beam` smallest are extracted with warp-wide
//            integer minimum reductions on (score bits | code) keys.
//   stage 2 (four targets x eight beam entries = 32 lanes): every lane takes one
//            (target, beam entry), forms its residual r = t - c1 and streams all of
//            codebook 2 from shared memory (broadcast loads of codeword pairs):
//            score2 = ||r||^2/2 + ||c2||^2/2 - <r, c2>, 8 packed FMAs per pair of
//            codewords, one three-input min; only the minimum of each 32-codeword
//            sub-chunk is kept.
//   decision: the eight lanes of a target agree on the smallest score; sub-chunks
//            within the rounding-error margin of it are revisited and the
//            codewords within the margin get their binary64 distance.
// Fast scores are binary32.  Every decision they cannot settle within twice their
// rounding-error bound (membership of the beam, the final argmin) is taken on
// binary64 distances accumulated in index order, so the result is the argmin of
// (distance, code1, code2) over the pool exactly as defined.
#include <cuda_fp16.h>

#include "pvt_internal.h"

namespace pvt {

// header + the image of the codebooks (two codebooks: under 40 KiB; up to four: under 56 KiB)
size_t encode_m2_workspace_bytes() { return kWsHeaderBytes + 57344; }

namespace {

constexpr int kM2Threads = 256;
constexpr int kM2CtasPerSm = 3;  // resident CTAs per SM the kernel is compiled for (registers) and launched as
constexpr int kM2K = 256;  // codebooks are padded to this many codewords
constexpr float kPadHalfNorm = 3.0e38f;
constexpr float kInf = __builtin_huge_valf();

struct EncM2Params {
  const float* W;
  const float* g;
  const float* scale;
  const uint32_t* idx;
  uint64_t k, G;
  uint32_t gpr;
  float eta;
  const void* books;
  int cb_f16;
  uint32_t K, beam;
  uint16_t* codes;  // two adjacent bytes per group
  float* err_out;
  uint32_t* status;
};

constexpr int kM2Group = 4;  // targets per warp iteration: 4 targets x 8 beam entries = 32 lanes

// Everything the kernel derives from the two codebooks, in the byte order it has in shared memory.  One small
// kernel writes it once per call into the workspace; every CTA of the search fetches it with a single bulk copy
// (cp.async.bulk, completion on an mbarrier; no multicast).
struct M2Image {
  alignas(16) float c1[kM2K][8];
  alignas(16) float c2[kM2K][8];
  alignas(16) uint64_t p1[4][8][32];  // stage-1 operands: (c1[l+64q][i], c1[l+64q+32][i])
  uint64_t h1[4][32];                 // (||c1||^2/2) pairs in the same order
  union {
    struct {
      alignas(16) float x2[kM2K / 2][16];  // FP32 stage 2: pair p holds (c2[2p][0], c2[2p+1][0], c2[2p][1], ...)
      alignas(8) float hx2[kM2K / 2][2];   // (||c2||^2/2) of the pair
    };
    // tensor stage 2: B fragments of codebook 2, word [n-tile][lane] = halves (c2[8 nt + lane/4][2 (lane%4)], [.. + 1])
    uint32_t b2[kM2K / 8][32];
  };
  alignas(8) float h2[kM2K];
  float n1max, n2max;
  float pad_[2];
};
static_assert(sizeof(M2Image) % 16 == 0, "the bulk copy moves multiples of 16 bytes");

struct M2Smem {
  M2Image img;
  // the sub-chunk minima of a warp's 32 residual rows on their way to the lanes that own the rows (tensor stage 2)
  alignas(16) float wmin[kM2Threads / 32][32][8];
  alignas(16) float wt[kM2Threads / 32][kM2Group][8];     // the targets of a warp's group
  alignas(16) uint32_t wk[kM2Threads / 32][kM2Group][8];  // their beam entries (codes of codebook 1)
  alignas(8) uint64_t img_bar;                            // completion of the image copy
};

__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float min3(float a, float b, float c) {
  float d;
  asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// D = A (16 x 16, rows = residuals) x B (16 x 8, columns = codewords) + C, fp16 operands, fp32 accumulation
__device__ __forceinline__ void mma_16x8x16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1, float c0,
                                            float c1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%10, %11, %10, %11};"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(c0), "f"(c1));
}
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  return (uint64_t)__float_as_uint(lo) | ((uint64_t)__float_as_uint(hi) << 32);
}
__device__ __forceinline__ float lo_of(uint64_t v) { return __uint_as_float((uint32_t)v); }
__device__ __forceinline__ float hi_of(uint64_t v) { return __uint_as_float((uint32_t)(v >> 32)); }
// order-preserving map binary32 -> u32
__device__ __forceinline__ uint32_t ord(float f) {
  const uint32_t b = __float_as_uint(f);
  return b ^ ((b >> 31) ? 0xffffffffu : 0x80000000u);
}
__device__ __forceinline__ float unord(uint32_t o) {
  return __uint_as_float(o ^ ((o >> 31) ? 0x80000000u : 0xffffffffu));
}

// ||t - c||^2 in binary64, the operations of the definition in index order
__device__ __forceinline__ double exact1(const float* t, const float* c) {
  double d = 0.0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const double e = __dsub_rn((double)t[i], (double)c[i]);
    d = __dadd_rn(d, __dmul_rn(e, e));
  }
  return d;
}
// ||(t - c1) - c2||^2 in binary64, residual carried in binary64
__device__ __forceinline__ double exact2(const float* t, const float* c1, const float* c2) {
  double d = 0.0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const double r = __dsub_rn((double)t[i], (double)c1[i]);
    const double e = __dsub_rn(r, (double)c2[i]);
    d = __dadd_rn(d, __dmul_rn(e, e));
  }
  return d;
}

__device__ __forceinline__ float load_cb(const void* books, int f16, uint32_t m, uint32_t kappa, uint32_t K, int i) {
  const size_t off = ((size_t)m * K + kappa) * 8 + i;
  return f16 ? __half2float(reinterpret_cast<const __half*>(books)[off]) : reinterpret_cast<const float*>(books)[off];
}

// ---- PTX helpers of the image copy ----------------------------------------------------------------------------
constexpr uint32_t kM2MaxSpins = 1u << 22;  // polls after which the wait for the image gives up
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool mbar_try_wait0(uint32_t bar) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar)
      : "memory");
  return ok != 0;
}
// One bulk copy global -> shared of the whole image (16-byte aligned on both sides, a multiple of 16 bytes),
// issued by one thread; every thread then waits, a bounded number of polls, for its completion.  Returns false
// (after recording PVT_DEV_WAIT_EXPIRED) if the copy has not landed by then: the CTA must leave without reading it.
__device__ __forceinline__ bool fetch_image(void* dst, const void* src, uint32_t bytes, uint64_t* bar, uint32_t* status) {
  const uint32_t b = smem_addr(bar);
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(b));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(dst)),
                 "l"(src), "r"(bytes), "r"(b)
                 : "memory");
  }
  __syncthreads();  // the barrier is initialised before anybody polls it
  bool ok = false;
  for (uint32_t spin = 0; spin < kM2MaxSpins && !ok; ++spin) {
    ok = mbar_try_wait0(b);
    if (!ok && spin > 4096) __nanosleep(64);
  }
  if (!ok) atomicOr(status, PVT_DEV_WAIT_EXPIRED);
  // everybody agrees (a thread that gave up makes the whole CTA leave)
  return __syncthreads_and(ok) != 0;
}

// ---- the codebook image: one block, one codeword per thread (K <= 256 = block size) ----
// TC2: stage 2 on the tensor cores (fp16 codebooks: the codewords are exact halves), else on the FP32 pipe.
template <bool TC2>
__global__ void __launch_bounds__(kM2Threads) m2_image_kernel(const EncM2Params p, M2Image* __restrict__ img_out) {
  __shared__ float red[kM2Threads / 32][2];
  M2Image& sm = *img_out;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  {
    float c1[8], c2[8], n1 = 0.0f, n2 = 0.0f;
    const bool real = (uint32_t)tid < p.K;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      c1[i] = real ? load_cb(p.books, p.cb_f16, 0, tid, p.K, i) : 0.0f;
      c2[i] = real ? load_cb(p.books, p.cb_f16, 1, tid, p.K, i) : 0.0f;
      n1 = __fmaf_rn(c1[i], c1[i], n1);
      n2 = __fmaf_rn(c2[i], c2[i], n2);
      sm.c1[tid][i] = c1[i];
      sm.c2[tid][i] = c2[i];
    }
    const float h1 = real ? 0.5f * n1 : kPadHalfNorm, h2 = real ? 0.5f * n2 : kPadHalfNorm;
    // codeword tid = l + 32*jj, jj = 2q + half
    const int l = tid & 31, jj = tid >> 5, q = jj >> 1, half = jj & 1;
    float* p1f = reinterpret_cast<float*>(&sm.p1[0][0][0]);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      p1f[(((q * 8 + i) * 32) + l) * 2 + half] = c1[i];
      if (!TC2) sm.x2[tid >> 1][2 * i + (tid & 1)] = c2[i];
    }
    reinterpret_cast<float*>(&sm.h1[0][0])[(q * 32 + l) * 2 + half] = h1;
    if (TC2) {
#pragma unroll
      for (int qq = 0; qq < 4; ++qq) {
        const __half2 v = __floats2half2_rn(c2[2 * qq], c2[2 * qq + 1]);  // exact: the codebook is fp16
        sm.b2[tid >> 3][4 * (tid & 7) + qq] = *reinterpret_cast<const uint32_t*>(&v);
      }
    } else {
      sm.hx2[tid >> 1][tid & 1] = h2;
    }
    sm.h2[tid] = h2;
    float m1 = n1, m2 = n2;
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, o));
      m2 = fmaxf(m2, __shfl_xor_sync(0xffffffffu, m2, o));
    }
    if (lane == 0) {
      red[warp][0] = m1;
      red[warp][1] = m2;
    }
    __syncthreads();
    if (tid == 0) {
      float a = 0.0f, b = 0.0f;
      for (int w = 0; w < kM2Threads / 32; ++w) {
        a = fmaxf(a, red[w][0]);
        b = fmaxf(b, red[w][1]);
      }
      sm.n1max = a;
      sm.n2max = b;
      sm.pad_[0] = sm.pad_[1] = 0.0f;
    }
  }
}

template <bool TC2>
__global__ void __launch_bounds__(kM2Threads, kM2CtasPerSm) encode_m2_kernel(const EncM2Params p,
                                                                              const M2Image* __restrict__ image) {
  __shared__ M2Smem smem;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (!fetch_image(&smem.img, image, (uint32_t)sizeof(M2Image), &smem.img_bar, p.status)) return;
  M2Image& sm = smem.img;
  const float n1max = sm.n1max, n2max = sm.n2max;
  const float s1max = sqrtf(n1max), s2max = sqrtf(n2max);
  const uint32_t B = p.beam;  // already min(beam, K)

  const uint64_t nwarps = (uint64_t)gridDim.x * (kM2Threads / 32);
  const uint64_t n_groups = (p.k + kM2Group - 1) / kM2Group;
  const uint32_t my_q = (uint32_t)lane >> 3, my_b = (uint32_t)lane & 7u;

  for (uint64_t gi = (uint64_t)blockIdx.x * (kM2Threads / 32) + warp; gi < n_groups; gi += nwarps) {
    // what this lane needs of its own target (target my_q of the group)
    uint32_t my_j = 0xffffffffu, my_prev = 0;
    float my_margin2 = 0.0f;

    // the four targets of the group, one element per lane (lane = 8 * target + element): index, W, g, row scale
    // and previous pair are fetched for all four at once, one fma and one division per lane (binary32)
    uint32_t lane_j = 0xffffffffu, lane_prev = 0;
    {
      const uint64_t n_mine = gi * kM2Group + my_q;
      if (n_mine < p.k) lane_j = __ldg(p.idx + n_mine);
      float tv = 0.0f;
      if (lane_j < p.G) {
        const float wv = __ldg(p.W + (size_t)lane_j * 8 + my_b), gv = __ldg(p.g + (size_t)lane_j * 8 + my_b);
        const float sc = __ldg(p.scale + lane_j / p.gpr);
        lane_prev = p.codes[lane_j];
        tv = __fdiv_rn(__fmaf_rn(-p.eta, gv, wv), sc);
      }
      smem.wt[warp][my_q][my_b] = tv;
    }
    __syncwarp();

    // ---- stage 1, one target after the other, the whole warp on each
#pragma unroll 1
    for (uint32_t q = 0; q < (uint32_t)kM2Group; ++q) {
      const uint64_t n = gi * kM2Group + q;
      if (n >= p.k) break;
      const uint32_t j = __shfl_sync(0xffffffffu, lane_j, 8 * q);
      const uint32_t prev = __shfl_sync(0xffffffffu, lane_prev, 8 * q);
      if (j >= p.G) {
        if (lane == 0) atomicOr(p.status, PVT_DEV_BAD_INDEX);
        continue;
      }
      float t[8];
      {
        const float4 ta = *reinterpret_cast<const float4*>(&smem.wt[warp][q][0]);
        const float4 tb = *reinterpret_cast<const float4*>(&smem.wt[warp][q][4]);
        t[0] = ta.x, t[1] = ta.y, t[2] = ta.z, t[3] = ta.w, t[4] = tb.x, t[5] = tb.y, t[6] = tb.z, t[7] = tb.w;
      }
      float nt2 = 0.0f;
#pragma unroll
      for (int i = 0; i < 8; ++i) nt2 = fmaf(t[i], t[i], nt2);
      const float tnorm = sqrtf(nt2);
      // twice the rounding-error bounds of the two fast scores (factor >= 2 to spare), u = 2^-24:
      //   |score1_fl - score1| <= 16.1 u (||c1||^2/2 + ||t|| ||c1||)
      //   |score2_fl - score2| <= 26 u (||t|| + max||c1|| + max||c2||)^2
      const float margin1 = 3.8146973e-6f /* 2^-18 */ * (0.5f * n1max + tnorm * s1max) + 1e-30f;
      const float sall = tnorm + s1max + s2max;
      const float margin2 = 7.6293945e-6f /* 2^-17 */ * sall * sall + 1e-30f;

      // 256 scores, 8 per lane
      float f[8];
      {
        uint64_t acc[4];
#pragma unroll
        for (int qq = 0; qq < 4; ++qq) acc[qq] = sm.h1[qq][lane];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const uint64_t ntd = pack2(-t[i], -t[i]);
#pragma unroll
          for (int qq = 0; qq < 4; ++qq) acc[qq] = fma2(ntd, sm.p1[qq][i][lane], acc[qq]);
        }
#pragma unroll
        for (int qq = 0; qq < 4; ++qq) {
          f[2 * qq] = lo_of(acc[qq]);
          f[2 * qq + 1] = hi_of(acc[qq]);
        }
      }
      // extract the B smallest (score truncated to 24 bits | code): a first guess of the beam.  Every lane sorts
      // its eight keys once (19 compare-exchanges); a round is then one warp minimum of the lanes' heads and a shift
      // of the winning lane's list.
      uint32_t key[8];
#pragma unroll
      for (int jj = 0; jj < 8; ++jj) key[jj] = (ord(f[jj]) & 0xffffff00u) | (uint32_t)(lane + 32 * jj);
#define PVT_CE(a, b)                               \
  {                                                \
    const uint32_t lo_ = min(key[a], key[b]);      \
    key[b] = max(key[a], key[b]);                  \
    key[a] = lo_;                                  \
  }
      PVT_CE(0, 2) PVT_CE(1, 3) PVT_CE(4, 6) PVT_CE(5, 7)
      PVT_CE(0, 4) PVT_CE(1, 5) PVT_CE(2, 6) PVT_CE(3, 7)
      PVT_CE(0, 1) PVT_CE(2, 3) PVT_CE(4, 5) PVT_CE(6, 7)
      PVT_CE(2, 4) PVT_CE(3, 5)
      PVT_CE(1, 4) PVT_CE(3, 6)
      PVT_CE(1, 2) PVT_CE(3, 4) PVT_CE(5, 6)
#undef PVT_CE
      uint32_t beam_code[8];
      uint32_t last = 0;  // the key extracted last
#pragma unroll
      for (int b = 0; b < 8; ++b) {
        beam_code[b] = 0;
        if ((uint32_t)b < B) {
          last = __reduce_min_sync(0xffffffffu, key[0]);
          beam_code[b] = last & 0xffu;
          const bool own = key[0] == last;  // keys are distinct: they end in the code
#pragma unroll
          for (int jj = 0; jj < 7; ++jj) key[jj] = own ? key[jj + 1] : key[jj];
          key[7] = own ? 0xffffffffu : key[7];
        }
      }
      // is that guess provably the exact beam?  theta = an upper bound of the scores in the guess (the top of the
      // truncation bucket of the key extracted last); every member of the exact beam scores <= theta + margin1; if
      // exactly B codewords do, they are the guess and the exact beam at once.
      {
        uint32_t cnt = 0;
        const float theta = unord(last | 0xffu);
        const float limit1 = theta + margin1;
        uint32_t member = 0;
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
          const bool in = f[jj] <= limit1 && (uint32_t)(lane + 32 * jj) < p.K;
          member |= in ? (1u << jj) : 0u;
          cnt += in;
        }
        cnt = __reduce_add_sync(0xffffffffu, cnt);
        if (cnt != B) {
          // undecided: order the shortlisted codewords by (binary64 distance, code)
          for (uint32_t b = 0; b < B; ++b) {
            double ld = __longlong_as_double(0x7ff0000000000000ll);
            uint32_t lk = 0xffffffffu;
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) {
              if (member & (1u << jj)) {
                const uint32_t kap = lane + 32 * jj;
                const double d = exact1(t, sm.c1[kap]);
                if (d < ld || (d == ld && kap < lk)) {
                  ld = d;
                  lk = kap;
                }
              }
            }
            // warp-wide lexicographic minimum of (ld, lk); distances are >= 0 so their bits order like u64
            const uint64_t bits = (uint64_t)__double_as_longlong(ld);
            const uint32_t hi = (uint32_t)(bits >> 32), lo = (uint32_t)bits;
            const uint32_t mhi = __reduce_min_sync(0xffffffffu, hi);
            const uint32_t mlo = __reduce_min_sync(0xffffffffu, hi == mhi ? lo : 0xffffffffu);
            const uint32_t mk = __reduce_min_sync(0xffffffffu, (hi == mhi && lo == mlo) ? lk : 0xffffffffu);
            const uint32_t chosen = mk < kM2K ? mk : 0u;
#pragma unroll
            for (int bb = 0; bb < 8; ++bb)
              if ((uint32_t)bb == b) beam_code[bb] = chosen;
            if ((chosen & 31u) == (uint32_t)lane) member &= ~(1u << (chosen >> 5));
          }
        }
      }
      // hand the target and its beam to the lanes of stage 2
      if (lane == 0) {
        *reinterpret_cast<uint4*>(&smem.wk[warp][q][0]) = make_uint4(beam_code[0], beam_code[1], beam_code[2], beam_code[3]);
        *reinterpret_cast<uint4*>(&smem.wk[warp][q][4]) = make_uint4(beam_code[4], beam_code[5], beam_code[6], beam_code[7]);
      }
      if (my_q == q) {
        my_j = j;
        my_prev = prev;
        my_margin2 = margin2;
      }
    }
    __syncwarp();

    // ---- stage 2: lane = (target my_q, beam entry my_b) against all of codebook 2
    const bool active = my_j != 0xffffffffu && my_b < B;
    float t[8], c1v[8], r[8];
    uint32_t k1 = 0;
    {
      const float4 ta = *reinterpret_cast<const float4*>(&smem.wt[warp][my_q][0]);
      const float4 tb = *reinterpret_cast<const float4*>(&smem.wt[warp][my_q][4]);
      t[0] = ta.x; t[1] = ta.y; t[2] = ta.z; t[3] = ta.w; t[4] = tb.x; t[5] = tb.y; t[6] = tb.z; t[7] = tb.w;
      k1 = active ? smem.wk[warp][my_q][my_b] : 0u;
      const float4 ca = *reinterpret_cast<const float4*>(&sm.c1[k1][0]);
      const float4 cb = *reinterpret_cast<const float4*>(&sm.c1[k1][4]);
      c1v[0] = ca.x; c1v[1] = ca.y; c1v[2] = ca.z; c1v[3] = ca.w; c1v[4] = cb.x; c1v[5] = cb.y; c1v[6] = cb.z; c1v[7] = cb.w;
    }
    float rho = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      r[i] = active ? __fsub_rn(t[i], c1v[i]) : 0.0f;
      rho = __fmaf_rn(r[i], r[i], rho);
    }
    rho = __fmul_rn(0.5f, rho);
    float sub_min[8];
    if (TC2) {
      // The 32 residuals of the group are the rows of two 16-row A tiles, each row [ -hi(2^e r) | -lo(2^e r) ] in fp16
      // (hi + lo keeps 22 significant bits of r, or all bits above 2^-25 in scaled units); the columns of B are the
      // codewords of codebook 2, [ c2 | c2 ]; C starts at 2^e ||c2||^2/2.  e is common to the group: the largest
      // residual element becomes [1/2, 1).  A thread holds elements 2 qd, 2 qd + 1 of rows g8, g8 + 8 of each tile.
      const uint32_t g8 = (uint32_t)lane >> 2, qd = (uint32_t)lane & 3u;
      float2 nr[4];  // -r of the four rows of this thread
      float rmax = 0.0f;
#pragma unroll
      for (int r4 = 0; r4 < 4; ++r4) {
        const uint32_t row = 16u * (r4 >> 1) + 8u * (r4 & 1) + g8, tq = row >> 3, b = row & 7u;
        const uint32_t tj = __shfl_sync(0xffffffffu, my_j, 8 * tq);
        const bool valid = tj != 0xffffffffu && b < B;
        const uint32_t kr = valid ? smem.wk[warp][tq][b] : 0u;  // the beam of a skipped target was never written
        const float2 tt = *reinterpret_cast<const float2*>(&smem.wt[warp][tq][2 * qd]);
        const float2 cc = *reinterpret_cast<const float2*>(&sm.c1[kr][2 * qd]);
        nr[r4].x = valid ? __fsub_rn(cc.x, tt.x) : 0.0f;  // -(t - c1), exactly
        nr[r4].y = valid ? __fsub_rn(cc.y, tt.y) : 0.0f;
        rmax = fmaxf(rmax, fmaxf(fabsf(nr[r4].x), fabsf(nr[r4].y)));
      }
      const uint32_t rbits = __reduce_max_sync(0xffffffffu, __float_as_uint(rmax));  // non-negative floats order as u32
      int e = 126 - (int)((rbits >> 23) & 0xffu);
      e = e > 15 ? 15 : (e < -100 ? -100 : e);
      const float sc = __uint_as_float((uint32_t)(e + 127) << 23), inv = __uint_as_float((uint32_t)(127 - e) << 23);
      uint32_t a[2][4];
#pragma unroll
      for (int r4 = 0; r4 < 4; ++r4) {
        const float x = nr[r4].x * sc, y = nr[r4].y * sc;
        const __half2 hi = __floats2half2_rn(x, y);
        const float2 back = __half22float2(hi);
        const __half2 lo = __floats2half2_rn(x - back.x, y - back.y);
        a[r4 >> 1][r4 & 1] = *reinterpret_cast<const uint32_t*>(&hi);
        a[r4 >> 1][2 + (r4 & 1)] = *reinterpret_cast<const uint32_t*>(&lo);
      }
#pragma unroll 2
      for (int sub = 0; sub < 8; ++sub) {
        float m[4] = {kInf, kInf, kInf, kInf};
#pragma unroll
        for (int n4 = 0; n4 < 4; ++n4) {
          const int nt = 4 * sub + n4;
          const uint32_t b = sm.b2[nt][lane];
          const float2 hh = *reinterpret_cast<const float2*>(&sm.h2[8 * nt + 2 * qd]);
          const float hx = hh.x * sc, hy = hh.y * sc;
          float d0[4], d1[4];
          mma_16x8x16(d0, a[0], b, b, hx, hy);
          mma_16x8x16(d1, a[1], b, b, hx, hy);
          m[0] = min3(m[0], d0[0], d0[1]);
          m[1] = min3(m[1], d0[2], d0[3]);
          m[2] = min3(m[2], d1[0], d1[1]);
          m[3] = min3(m[3], d1[2], d1[3]);
        }
#pragma unroll
        for (int r4 = 0; r4 < 4; ++r4) {
          m[r4] = fminf(m[r4], __shfl_xor_sync(0xffffffffu, m[r4], 1));
          m[r4] = fminf(m[r4], __shfl_xor_sync(0xffffffffu, m[r4], 2));
        }
        if (qd == 0) {
#pragma unroll
          for (int r4 = 0; r4 < 4; ++r4) smem.wmin[warp][16 * (r4 >> 1) + 8 * (r4 & 1) + g8][sub] = m[r4];
        }
      }
      __syncwarp();
      {
        const float4 ma = *reinterpret_cast<const float4*>(&smem.wmin[warp][lane][0]);
        const float4 mb = *reinterpret_cast<const float4*>(&smem.wmin[warp][lane][4]);
        const float mm[8] = {ma.x, ma.y, ma.z, ma.w, mb.x, mb.y, mb.z, mb.w};
#pragma unroll
        for (int sub = 0; sub < 8; ++sub) sub_min[sub] = active ? __fmaf_rn(mm[sub], inv, rho) : kInf;
      }
      // the halves' absolute rounding floor (2^-25 per element in scaled units), doubled, with a factor 4 to spare
      my_margin2 += 4.76837158203125e-7f /* 2^-21 */ * inv * s2max;
    } else {
      uint64_t nrd[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) nrd[i] = pack2(-r[i], -r[i]);
      const uint64_t rho2 = pack2(rho, rho);
#pragma unroll
      for (int sub = 0; sub < 8; ++sub) {
        float cmin = kInf;
        const ulonglong2* vals = reinterpret_cast<const ulonglong2*>(&sm.x2[0][0]) + sub * 16 * 4;
        const uint64_t* norms = reinterpret_cast<const uint64_t*>(&sm.hx2[0][0]) + sub * 16;
#pragma unroll 4
        for (int pr = 0; pr < 16; ++pr) {
          const ulonglong2 q0 = vals[4 * pr], q1 = vals[4 * pr + 1], q2 = vals[4 * pr + 2], q3 = vals[4 * pr + 3];
          uint64_t acc = add2(norms[pr], rho2);
          acc = fma2(nrd[0], q0.x, acc);
          acc = fma2(nrd[1], q0.y, acc);
          acc = fma2(nrd[2], q1.x, acc);
          acc = fma2(nrd[3], q1.y, acc);
          acc = fma2(nrd[4], q2.x, acc);
          acc = fma2(nrd[5], q2.y, acc);
          acc = fma2(nrd[6], q3.x, acc);
          acc = fma2(nrd[7], q3.y, acc);
          cmin = min3(cmin, lo_of(acc), hi_of(acc));
        }
        sub_min[sub] = active ? cmin : kInf;
      }
    }
    float gmin = sub_min[0];
#pragma unroll
    for (int sub = 1; sub < 8; ++sub) gmin = fminf(gmin, sub_min[sub]);
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) gmin = fminf(gmin, __shfl_xor_sync(0xffffffffu, gmin, o));
    const float limit2 = gmin + my_margin2;

    // ---- decision in binary64 among the pairs within the margin, plus the previous pair.
    // The eight lanes of a target revisit its sub-chunks within the margin one after the other, four codewords per
    // lane, the four targets of the group side by side; every lane keeps the best (distance, code pair) it has seen.
    // (The fast score is evaluated again here, in another order: both evaluations lie within half the margin of the
    // true score, so the pair the definition selects passes both tests.)
    double bd = __longlong_as_double(0x7ff0000000000000ll);
    uint32_t bk = 0xffffffffu;  // code1 << 8 | code2: orders like (code1, code2)
    {
      uint32_t hm = 0;  // sub-chunks of this lane's beam entry within the margin
#pragma unroll
      for (int sub = 0; sub < 8; ++sub) hm |= (active && sub_min[sub] <= limit2) ? (1u << sub) : 0u;
      // the target's 64 (beam entry, sub-chunk) flags: byte b belongs to beam entry b
      uint32_t hlo = my_b < 4 ? hm << (8 * my_b) : 0u, hhi = my_b >= 4 ? hm << (8 * (my_b - 4)) : 0u;
#pragma unroll
      for (int o = 1; o < 8; o <<= 1) {
        hlo |= __shfl_xor_sync(0xffffffffu, hlo, o);
        hhi |= __shfl_xor_sync(0xffffffffu, hhi, o);
      }
      while (__any_sync(0xffffffffu, (hlo | hhi) != 0u)) {
        const bool work = (hlo | hhi) != 0u;
        uint32_t pos = 0;
        if (hlo) {
          pos = (uint32_t)__ffs(hlo) - 1u;
          hlo &= hlo - 1u;
        } else if (hhi) {
          pos = 32u + (uint32_t)__ffs(hhi) - 1u;
          hhi &= hhi - 1u;
        }
        const uint32_t hb = pos >> 3, hsub = pos & 7u;
        const uint32_t hk1 = work ? smem.wk[warp][my_q][hb] : 0u;
        float sc1[8], sr[8], srho = 0.0f;
        {
          const float4 ca = *reinterpret_cast<const float4*>(&sm.c1[hk1][0]);
          const float4 cb = *reinterpret_cast<const float4*>(&sm.c1[hk1][4]);
          sc1[0] = ca.x; sc1[1] = ca.y; sc1[2] = ca.z; sc1[3] = ca.w;
          sc1[4] = cb.x; sc1[5] = cb.y; sc1[6] = cb.z; sc1[7] = cb.w;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          sr[i] = __fsub_rn(t[i], sc1[i]);
          srho = __fmaf_rn(sr[i], sr[i], srho);
        }
        srho = __fmul_rn(0.5f, srho);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const uint32_t k2 = hsub * 32u + 8u * c + my_b;
          float c2v[8];
          {
            const float4 ca = *reinterpret_cast<const float4*>(&sm.c2[k2][0]);
            const float4 cb = *reinterpret_cast<const float4*>(&sm.c2[k2][4]);
            c2v[0] = ca.x; c2v[1] = ca.y; c2v[2] = ca.z; c2v[3] = ca.w;
            c2v[4] = cb.x; c2v[5] = cb.y; c2v[6] = cb.z; c2v[7] = cb.w;
          }
          float s2 = __fadd_rn(sm.h2[k2], srho);
#pragma unroll
          for (int i = 0; i < 8; ++i) s2 = __fmaf_rn(-sr[i], c2v[i], s2);
          if (work && s2 <= limit2 && k2 < p.K) {
            const double d = exact2(t, sc1, c2v);
            const uint32_t kk = (hk1 << 8) | k2;
            if (d < bd || (d == bd && kk < bk)) {
              bd = d;
              bk = kk;
            }
          }
        }
      }
    }
    if (my_b == 0 && my_j != 0xffffffffu) {  // the previous pair joins the pool
      const uint32_t q1 = my_prev & 0xffu, q2 = my_prev >> 8;
      if (q1 < p.K && q2 < p.K) {
        const double d = exact2(t, sm.c1[q1], sm.c2[q2]);
        const uint32_t kk = (q1 << 8) | q2;
        if (d < bd || (d == bd && kk < bk)) {
          bd = d;
          bk = kk;
        }
      } else {
        atomicOr(p.status, PVT_DEV_BAD_CODE);
      }
    }
    // lexicographic minimum of (bd, bk) over the eight lanes of the target
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) {
      const uint64_t bits = (uint64_t)__double_as_longlong(bd);
      const uint32_t ohi = __shfl_xor_sync(0xffffffffu, (uint32_t)(bits >> 32), o);
      const uint32_t olo = __shfl_xor_sync(0xffffffffu, (uint32_t)bits, o);
      const uint32_t ok = __shfl_xor_sync(0xffffffffu, bk, o);
      const double od = __longlong_as_double((long long)(((uint64_t)ohi << 32) | olo));
      if (od < bd || (od == bd && ok < bk)) {
        bd = od;
        bk = ok;
      }
    }
    if (my_b == 0 && my_j != 0xffffffffu && bk != 0xffffffffu) {
      p.codes[my_j] = (uint16_t)(((bk >> 8) & 0xffu) | ((bk & 0xffu) << 8));
      if (p.err_out) p.err_out[gi * kM2Group + my_q] = (float)bd;
    }
    __syncwarp();  // the group's scratch is rewritten by the next iteration
  }
}

}  // namespace

cudaError_t launch_encode_m2(const pvt_layer& L, uint64_t G, const uint32_t* idx, uint64_t k, float* err_out,
                             void* ws, int sm_count, cudaStream_t stream) {
  EncM2Params p;
  p.W = L.W;
  p.g = L.g;
  p.scale = L.scale;
  p.idx = idx;
  p.k = k;
  p.G = G;
  p.gpr = (uint32_t)(L.cols / kGroupDim);
  p.eta = L.eta;
  p.books = L.codebooks;
  p.cb_f16 = L.codebook_dtype == PVT_F16;
  p.K = (uint32_t)L.codebook_size;
  p.beam = (uint32_t)L.beam < p.K ? (uint32_t)L.beam : p.K;
  p.codes = reinterpret_cast<uint16_t*>(L.codes);
  p.err_out = err_out;
  p.status = reinterpret_cast<uint32_t*>(ws);
  const uint64_t warps_per_cta = kM2Threads / 32;
  const uint64_t groups = (k + kM2Group - 1) / kM2Group;
  uint64_t ctas = (groups + warps_per_cta - 1) / warps_per_cta;
  if (ctas > kM2CtasPerSm * (uint64_t)sm_count) ctas = kM2CtasPerSm * (uint64_t)sm_count;  // persistent: the resident CTAs
  static_assert(sizeof(M2Image) <= 40960, "the workspace reserves 40 KiB for the image");
  M2Image* image = reinterpret_cast<M2Image*>(static_cast<char*>(ws) + kWsHeaderBytes);
  timing_begin(kKernEncodeAux, stream);
  if (p.cb_f16)
    m2_image_kernel<true><<<1, kM2Threads, 0, stream>>>(p, image);
  else
    m2_image_kernel<false><<<1, kM2Threads, 0, stream>>>(p, image);
  timing_end(kKernEncodeAux, stream);
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  timing_begin(kKernEncodeMain, stream);
  if (p.cb_f16)
    encode_m2_kernel<true><<<(unsigned)ctas, kM2Threads, 0, stream>>>(p, image);
  else
    encode_m2_kernel<false><<<(unsigned)ctas, kM2Threads, 0, stream>>>(p, image);
  count_launches(2);
  timing_end(kKernEncodeMain, stream);
  return cudaGetLastError();
}

}  // namespace pvt
