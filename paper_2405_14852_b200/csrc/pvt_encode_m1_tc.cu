// Exhaustive nearest-codeword search of the V step for one fp16 codebook on the
// tensor cores (Appendix C / Appendix J: all codewords of the codebook are tried;
// Appendix D: the score ||c||^2 - 2 <t, c>; Eq. 8 for the target).
//
// The score matrix S[n][kappa] = 2^e_n (<t_n, c_kappa> - ||c_kappa||^2 / 2) is a
// dense contraction of depth 8 (+ the norm term): it is evaluated tile by tile
// with tcgen05.mma (fp16 operands, fp32 accumulators in tensor memory) and never
// leaves the SM -- the epilogue reads each accumulator row once and keeps only
// its running maximum and the 64-codeword sub-chunks that come within an error
// margin of it.  The exact decision (binary64 distances, argmin of (distance,
// code)) is taken afterwards by the rescoring kernel on those sub-chunks, so the
// fp16 rounding of the operands only has to be bounded, not small.
//
// Operands (16-byte K chunks of 8 halves, no swizzle, K-major "interleaved" core-matrix
// layout: 8 rows x 16 bytes per core matrix, K chunks 128 bytes apart, 8-row groups of
// A 512 and of B 256 bytes apart; one MMA instruction consumes two K chunks, so a step is
// two instructions per A block, the second accumulating onto the first):
//   A row n     = [ hi_0 .. hi_7 | 2^e x 8 | lo_0 .. lo_7 | 0 x 8 ]
//                 hi_i = fp16(2^e t_i), lo_i = fp16(2^e t_i - hi_i)
//   B row kappa = [ c_0 .. c_7   | -h_hi, -h_lo, -h_lo2, 0 x 5 ]
//                 h = ||c||^2/2 = h_hi + h_lo + h_lo2
//   instruction 1: A chunks 0-1 x B chunks 0-1 (hi . c - 2^e h);  instruction 2: A chunks 2-3 x
//   the same B chunks (lo . c + 0): the codeword is stored and streamed once.
// Splitting t into two halves keeps 22 of its 24 significant bits, so the fast
// score is about as accurate as a binary32 evaluation and very few sub-chunks
// come within the margin.  The codebook image is written once per call by a small
// kernel in exactly the shared-memory byte order, so every 128-codeword step
// arrives with one 1-D bulk copy (4 KB); the A rows are written by the threads
// that own the targets.  e_n is chosen per target so that max_i |2^e t_i| lies in
// [1/2, 1).
//
// CTA = 256 targets (two 128-row A blocks) x a slice of the codebook, one CTA per
// SM, persistent over (tile, slice) units.  Warps 0-7: own one target per thread,
// build A, run the epilogue (warp w reads tensor-memory lanes 32 (w % 4) .. of the
// accumulator of A block w / 4).  Warp 8: bulk-copy producer (two stages of eight steps).
// Warps 9 and 10: each runs the issue loop of one A block as a whole warp (so that
// descriptors and addresses are warp-uniform values) with one lane issuing the MMAs;
// warp 9 also allocates tensor memory.  Tensor memory: 2 buffers x 2 accumulators x
// 128 columns = 512 columns, so the MMAs of step i+1 overlap the epilogue of step i.
// The pace is set by fixed costs per hand-over of an accumulator (issue -> execute ->
// completion seen -> read out -> release seen), not by a pipe: a wait on an mbarrier
// costs 100-150 cycles even on a finished phase, an MMA or a commit about 50, a
// tensor-memory load about 100 while MMAs are writing, and a thread that runs alone
// in divergent code pays several cycles per dependent instruction.  Hence: converged
// issue loops with constant parities and offsets, every result asked for well before
// it is used, and as few barrier operations per step as possible.
//
// Codewords whose half squared norm exceeds the fp16 range get a sentinel row
// that can never win and are listed as "exceptions": the rescoring kernel always
// evaluates them exactly.  Targets outside the range the scaling can serve
// (non-finite, or max |t_i| >= 256) are rescored against the whole codebook.
//
// Groups of 16 weights (Appendix J) use the same kernel with A rows of 48 halves, [ hi x 16 | lo x 16 | 2^e x 8 |
// 0 x 8 ], against B rows of 32 halves, [ c x 16 | norm terms | 0 x 8 ]: three instructions per step and A block
// (hi . c, lo . c, 2^e x norm terms), 8 KB per step.  Everything described for eight weights above holds with
// these sizes.
#include <atomic>

#include "pvt_encode_m1.cuh"

namespace pvt {

using namespace m1;

namespace {

constexpr int kTcTile = 256;            // targets per CTA tile
constexpr int kTcStepCw = 128;          // codewords per MMA step (the N of one instruction)
// Operand geometry for groups of DG weights.  The codeword appears once per row of the codebook image; the two
// halves of the target meet it in separate instructions that read the same K chunks of B:
//   DG = 8:   A row = [ hi | 2^e x 8 | lo | 0 ]  (4 chunks),  B row = [ c | norm terms ]  (2 chunks)
//             instruction 0: A chunks 0-1 x B chunks 0-1;  instruction 1: A chunks 2-3 x B chunks 0-1
//   DG = 16:  A row = [ hi x 16 | lo x 16 | 2^e x 8 | 0 ]  (6 chunks),  B row = [ c x 16 | norm terms | 0 ]  (4 chunks)
//             instructions: A 0-1 x B 0-1, A 2-3 x B 0-1, A 4-5 x B 2-3
template <int DG>
struct TcDim {
  static constexpr int kARowBytes = 2 * (2 * DG + 16);         // 64 or 96
  static constexpr int kAGroupBytes = 8 * kARowBytes;          // one 8-row group of A
  static constexpr int kABlockBytes = 128 * kARowBytes;        // one A block of 128 targets
  static constexpr int kBRowBytes = DG == 8 ? 32 : 64;
  static constexpr int kBGroupBytes = 8 * kBRowBytes;
  static constexpr int kStepBytes = kTcStepCw * kBRowBytes;    // codebook image per step: 4096 or 8192
  static constexpr int kMmas = DG == 8 ? 2 : 3;                // instructions per step and A block
  static constexpr int kPart = DG / 8;                         // K chunks per codeword
  // K chunk at which instruction m starts reading A and B
  __host__ __device__ static constexpr int a_chunk(int m) { return 2 * m; }
  __host__ __device__ static constexpr int b_chunk(int m) { return (DG == 16 && m == 2) ? 2 : 0; }
};
constexpr int kTcStepBytes = TcDim<8>::kStepBytes;
constexpr int kTcSubCw = 64;            // tracking granularity of the running maximum
constexpr int kTcGroupSteps = 8;        // steps per codebook stage: the MMA warps wait for the codebook once per eight steps
constexpr int kTcStages = 2;            // codebook stages (eight steps each: 32 KB, or 64 KB for groups of 16)
constexpr int kTcEpiThreads = 256;
constexpr int kTcThreads = kTcEpiThreads + 96;  // + producer warp + one MMA warp per A block
constexpr uint32_t kTmemCols = 512;
constexpr float kMaxHalfNorm = 60000.0f;  // largest ||c||^2/2 the image represents
constexpr float kNegInf = -__builtin_huge_valf();

}  // namespace

namespace {
std::atomic<int> g_m1_search{PVT_M1_AUTO};
std::atomic<uint32_t> g_max_spins{m1::kMaxSpins};
std::atomic<uint32_t> g_withhold_copy{m1::kNoWithhold};
}

namespace m1 {
WaitTestHook wait_test_hook() {
  return WaitTestHook{g_max_spins.load(std::memory_order_relaxed), g_withhold_copy.load(std::memory_order_relaxed)};
}
void set_wait_test_hook(uint32_t max_spins, uint32_t withhold_copy) {
  g_max_spins.store(max_spins, std::memory_order_relaxed);
  g_withhold_copy.store(withhold_copy, std::memory_order_relaxed);
}
}  // namespace m1

void set_m1_search(int mode) { g_m1_search.store(mode, std::memory_order_relaxed); }

bool encode_m1_use_tc(const pvt_layer& L, uint64_t k) {
  (void)k;
  if (L.num_codebooks != 1 || L.codebook_dtype != PVT_F16) return false;  // the operand image is fp16
  const int mode = g_m1_search.load(std::memory_order_relaxed);
  if (mode == PVT_M1_FP32) return false;
  if (mode == PVT_M1_TENSOR) return true;
  return L.codebook_size >= 1024;  // below that the FP32 pipe with its larger target tiles is as fast
}

EncodeM1TcLayout encode_m1_tc_layout(uint32_t K, uint64_t k, int sm_count, int group_dim) {
  EncodeM1TcLayout e;
  e.n_steps = (K + kTcStepCw - 1) / kTcStepCw;
  e.n_tiles = (uint32_t)((k + kTcTile - 1) / kTcTile);
  uint32_t best_s = 1;
  double best_eff = 0.0;
  // a slice should keep at least 16 steps so that building A stays a small part of a unit
  uint32_t s_max = e.n_steps / 16;
  if (s_max < 1) s_max = 1;
  if (s_max > (uint32_t)kMaxSlices) s_max = (uint32_t)kMaxSlices;
  for (uint32_t s = 1; s <= s_max; ++s) {
    const uint64_t units = (uint64_t)e.n_tiles * s;
    const uint64_t rounds = (units + sm_count - 1) / sm_count;
    const double eff = (double)units / (double)(rounds * sm_count);
    if (eff > best_eff + 0.03) {
      best_eff = eff;
      best_s = s;
    }
  }
  e.n_slices = best_s;
  const uint64_t units = (uint64_t)e.n_tiles * e.n_slices;
  e.n_ctas = (uint32_t)(units < (uint64_t)sm_count ? units : (uint64_t)sm_count);
  e.bimg_off = kWsHeaderBytes;
  e.stats_off = align_up(e.bimg_off + (size_t)e.n_steps * (group_dim == 16 ? TcDim<16>::kStepBytes : kTcStepBytes),
                         kWsAlign);
  e.exc_off = e.stats_off + kWsAlign;
  e.gbest_off = align_up(e.exc_off + sizeof(uint32_t) * K, kWsAlign);
  e.margin_off = align_up(e.gbest_off + sizeof(uint32_t) * k, kWsAlign);
  e.rec_off = align_up(e.margin_off + sizeof(float) * k, kWsAlign);
  e.bytes = align_up(e.rec_off + (size_t)e.n_tiles * e.n_slices * kTcTile * sizeof(CandRecord), kWsAlign);
  return e;
}

namespace {

// stats block in the workspace: [0] bit pattern of max ||c||^2 over representable codewords, [1] exception count
struct TcStats {
  uint32_t n2max_bits;
  uint32_t exc_count;
};

// ---- codebook image ------------------------------------------------------------
template <int DG>
__global__ void __launch_bounds__(256) tc_prep_kernel(const uint4* __restrict__ book, uint32_t K, uint32_t n_steps,
                                                       unsigned char* __restrict__ bimg, TcStats* stats,
                                                       uint32_t* __restrict__ exc_list) {
  using D = TcDim<DG>;
  const uint32_t kappa = blockIdx.x * blockDim.x + threadIdx.x;
  uint32_t n2bits = 0;
  if (kappa < n_steps * kTcStepCw) {
    const bool real = kappa < K;
    uint4 raw[D::kPart];
    float n2 = 0.0f;
#pragma unroll
    for (int part = 0; part < D::kPart; ++part) {
      raw[part] = make_uint4(0, 0, 0, 0);
      if (real) {
        raw[part] = __ldg(book + (size_t)kappa * D::kPart + part);
        const __half2* h = reinterpret_cast<const __half2*>(&raw[part]);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f = __half22float2(h[i]);
          n2 = __fmaf_rn(f.x, f.x, n2);
          n2 = __fmaf_rn(f.y, f.y, n2);
        }
      }
    }
    const float hn = 0.5f * n2;
    const bool rep = real && (hn <= kMaxHalfNorm);  // false for NaN / Inf as well
    if (real && !rep) {
      const uint32_t pos = atomicAdd(&stats->exc_count, 1u);
      if (pos < K) exc_list[pos] = kappa;
    }
    uint4 k1;
    if (rep) {
      const __half h_hi = __float2half_rn(hn);
      const float r1 = hn - __half2float(h_hi);
      const __half h_lo = __float2half_rn(r1);
      const float r2 = r1 - __half2float(h_lo);
      const __half h_lo2 = __float2half_rn(r2);
      const __half2 a = __halves2half2(__hneg(h_hi), __hneg(h_lo));
      const __half2 b = __halves2half2(__hneg(h_lo2), __float2half_rn(0.0f));
      k1 = make_uint4(*reinterpret_cast<const uint32_t*>(&a), *reinterpret_cast<const uint32_t*>(&b), 0u, 0u);
      n2bits = __float_as_uint(n2);
    } else {
      // padding and exceptions: zero codeword with the most negative norm terms, never a maximum
#pragma unroll
      for (int part = 0; part < D::kPart; ++part) raw[part] = make_uint4(0, 0, 0, 0);
      k1 = make_uint4(0xfbfffbffu, 0xfbfffbffu, 0xfbfffbffu, 0xfbfffbffu);  // -65504 x 8
    }
    const uint32_t step = kappa / kTcStepCw, r = kappa % kTcStepCw;
    unsigned char* row = bimg + (size_t)step * D::kStepBytes + (r >> 3) * D::kBGroupBytes + (r & 7) * 16;
#pragma unroll
    for (int part = 0; part < D::kPart; ++part) *reinterpret_cast<uint4*>(row + 128 * part) = raw[part];
    *reinterpret_cast<uint4*>(row + 128 * D::kPart) = k1;  // norm terms
    if (DG == 16) *reinterpret_cast<uint4*>(row + 128 * (D::kPart + 1)) = make_uint4(0, 0, 0, 0);
  }
  n2bits = __reduce_max_sync(0xffffffffu, n2bits);
  if ((threadIdx.x & 31) == 0 && n2bits > __ldcg(&stats->n2max_bits)) atomicMax(&stats->n2max_bits, n2bits);
}

// ---- tcgen05 wrappers -----------------------------------------------------------
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, fp16 x fp16 -> fp32, M = 128, N = 128, K = 16;
// accumulate == 0 overwrites D
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                         uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on the mbarrier once all MMAs issued so far by this thread have completed
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// shared-memory operand descriptor: K-major, no swizzle, K chunks 128 B apart, 8-row groups group_bytes apart
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t group_bytes) {
  return (uint64_t)((saddr & 0x3ffffu) >> 4) | ((uint64_t)(128u >> 4) << 16) |
         ((uint64_t)(group_bytes >> 4) << 32) | (1ull << 46);
}
// instruction descriptor: D fp32, A and B fp16, both K-major, N = 128, M = 128
constexpr uint32_t kIdesc = (1u << 4) | ((uint32_t)(kTcStepCw >> 3) << 17) | ((128u >> 4) << 24);

// 32 lanes x 64 consecutive columns of 32-bit accumulators -> 64 registers per thread
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, uint32_t* v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x64.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, "
      "%32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, "
      "%48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31]), "=r"(v[32]),
        "=r"(v[33]), "=r"(v[34]), "=r"(v[35]), "=r"(v[36]), "=r"(v[37]), "=r"(v[38]), "=r"(v[39]), "=r"(v[40]),
        "=r"(v[41]), "=r"(v[42]), "=r"(v[43]), "=r"(v[44]), "=r"(v[45]), "=r"(v[46]), "=r"(v[47]), "=r"(v[48]),
        "=r"(v[49]), "=r"(v[50]), "=r"(v[51]), "=r"(v[52]), "=r"(v[53]), "=r"(v[54]), "=r"(v[55]), "=r"(v[56]),
        "=r"(v[57]), "=r"(v[58]), "=r"(v[59]), "=r"(v[60]), "=r"(v[61]), "=r"(v[62]), "=r"(v[63])
      : "r"(taddr)
      : "memory");
}
// Wait for the outstanding tensor-memory loads.  The registers are passed through the
// statement so that no use of them can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_ld_wait(uint32_t* v) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
                 "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]),
                 "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]),
                 "+r"(v[23]), "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]),
                 "+r"(v[30]), "+r"(v[31]), "+r"(v[32]), "+r"(v[33]), "+r"(v[34]), "+r"(v[35]), "+r"(v[36]),
                 "+r"(v[37]), "+r"(v[38]), "+r"(v[39]), "+r"(v[40]), "+r"(v[41]), "+r"(v[42]), "+r"(v[43]),
                 "+r"(v[44]), "+r"(v[45]), "+r"(v[46]), "+r"(v[47]), "+r"(v[48]), "+r"(v[49]), "+r"(v[50]),
                 "+r"(v[51]), "+r"(v[52]), "+r"(v[53]), "+r"(v[54]), "+r"(v[55]), "+r"(v[56]), "+r"(v[57]),
                 "+r"(v[58]), "+r"(v[59]), "+r"(v[60]), "+r"(v[61]), "+r"(v[62]), "+r"(v[63])
               :
               : "memory");
}

// non-blocking test of a phase (try_wait may suspend the thread for a while when the phase is not complete)
__device__ __forceinline__ uint32_t mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float max64(const uint32_t* v) {
  float m0 = max3(__uint_as_float(v[0]), __uint_as_float(v[1]), __uint_as_float(v[2]));
  float m1 = max3(__uint_as_float(v[3]), __uint_as_float(v[4]), __uint_as_float(v[5]));
  float m2 = max3(__uint_as_float(v[6]), __uint_as_float(v[7]), __uint_as_float(v[8]));
  float m3 = max3(__uint_as_float(v[9]), __uint_as_float(v[10]), __uint_as_float(v[11]));
#pragma unroll
  for (int i = 12; i < 60; i += 8) {
    m0 = max3(m0, __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
    m1 = max3(m1, __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
    m2 = max3(m2, __uint_as_float(v[i + 4]), __uint_as_float(v[i + 5]));
    m3 = max3(m3, __uint_as_float(v[i + 6]), __uint_as_float(v[i + 7]));
  }
  m0 = max3(m0, __uint_as_float(v[60]), __uint_as_float(v[61]));
  m1 = max3(m1, __uint_as_float(v[62]), __uint_as_float(v[63]));
  return fmaxf(max3(m0, m1, m2), m3);
}

// ---- shared memory -----------------------------------------------------------------
template <int DG>
struct TcSmem {
  alignas(128) unsigned char a[2][TcDim<DG>::kABlockBytes];  // two A blocks of 128 targets
  alignas(128) unsigned char b[kTcStages][kTcGroupSteps][TcDim<DG>::kStepBytes];
  alignas(8) uint64_t full_bar[kTcStages];
  uint64_t empty_bar[kTcStages];
  uint64_t tmem_full[2][2];   // per buffer and A block
  uint64_t tmem_empty[2][2];
  uint64_t a_ready;
  uint64_t drain_bar[2];
  float list_max[kListLen][kTcTile];
  uint16_t list_id[kListLen][kTcTile];
  uint32_t tmem_base;
  uint32_t abort_flag;
};

// (The bound is the launch size itself: with 384 the register limit drops from 184 to 168, which the epilogue loop
// needs in full, and the same source runs 18 % slower.)
template <int DG>
__global__ void __launch_bounds__(kTcThreads, 1) encode_m1_tc_kernel(const EncM1Params p,
                                                                      const unsigned char* __restrict__ bimg,
                                                                      const TcStats* __restrict__ stats) {
  using D = TcDim<DG>;
  constexpr int kStepBytes = D::kStepBytes;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  TcSmem<DG>& sm = *reinterpret_cast<TcSmem<DG>*>(smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  volatile uint32_t* abort_flag = &sm.abort_flag;

  if (tid == 0) {
    sm.abort_flag = 0;
    for (int s = 0; s < kTcStages; ++s) {
      mbar_init(smem_u32(&sm.full_bar[s]), 1);
      mbar_init(smem_u32(&sm.empty_bar[s]), 2);  // one commit per MMA warp, at the stage's last step
    }
    for (int b = 0; b < 2; ++b) {
      for (int q = 0; q < 2; ++q) {
        mbar_init(smem_u32(&sm.tmem_full[b][q]), 1);
        mbar_init(smem_u32(&sm.tmem_empty[b][q]), kTcEpiThreads / 2);  // every thread of the block's four warps
      }
    }
    mbar_init(smem_u32(&sm.a_ready), kTcEpiThreads);
    mbar_init(smem_u32(&sm.drain_bar[0]), 1);
    mbar_init(smem_u32(&sm.drain_bar[1]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 9) {
    tmem_alloc(smem_u32(&sm.tmem_base), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&sm.tmem_base);

  const uint64_t units = (uint64_t)p.n_tiles * p.n_slices;

  if (warp == 8) {
    // ------------------------------------------------------------ bulk-copy producer
    // (the whole warp runs the loop, lane 0 issues the copies: no lane waits at the final barrier meanwhile)
    {
      // total number of steps of this CTA (for the byte count of the last, partial stage)
      uint32_t total = 0;
      for (uint64_t u = blockIdx.x; u < units; u += gridDim.x) {
        uint32_t s_lo, s_hi;
        slice_units(p, (uint32_t)(u % p.n_slices), &s_lo, &s_hi);
        total += s_hi - s_lo;
      }
      uint32_t it = 0;
      bool alive = true;
      for (uint64_t u = blockIdx.x; u < units && alive; u += gridDim.x) {
        uint32_t s_lo, s_hi;
        slice_units(p, (uint32_t)(u % p.n_slices), &s_lo, &s_hi);
        for (uint32_t st = s_lo; st < s_hi && alive; ++st, ++it) {
          const uint32_t grp = it / kTcGroupSteps, sub = it % kTcGroupSteps, s = grp % kTcStages;
          const uint32_t fb = smem_u32(&sm.full_bar[s]);
          if (sub == 0) {
            if (grp >= (uint32_t)kTcStages) {
              const uint32_t eb = smem_u32(&sm.empty_bar[s]), ep = ((grp / kTcStages) - 1) & 1;
              if (!__all_sync(0xffffffffu, mbar_try_wait(eb, ep))) {
                bool ok = true;
                if (lane == 0) ok = mbar_wait(eb, ep, abort_flag, p.status, p.max_spins);
                alive = __shfl_sync(0xffffffffu, ok, 0);
              }
            }
            if (!alive) break;
            const uint32_t left = total - it;
            if (lane == 0)
              mbar_expect_tx(fb, (left < (uint32_t)kTcGroupSteps ? left : (uint32_t)kTcGroupSteps) * kStepBytes);
            __syncwarp();
          }
          // test hook: a step that is never copied leaves its stage's barrier incomplete, so the MMA warps' wait
          // for that stage runs out
          if (lane == 0 && it != p.withhold_copy)
            bulk_g2s(smem_u32(&sm.b[s][sub][0]), bimg + (size_t)st * kStepBytes, kStepBytes, fb);
        }
      }
      if (!alive && lane == 0) {
        // let every copy that was issued land before the CTA may exit
        const uint32_t groups = (it + kTcGroupSteps - 1) / kTcGroupSteps;
        for (uint32_t back = 1; back <= (uint32_t)kTcStages && back <= groups; ++back) {
          const uint32_t j = groups - back;
          if (p.withhold_copy / kTcGroupSteps == j) continue;  // incomplete on purpose; its other copies landed long ago
          const uint32_t fb = smem_u32(&sm.full_bar[j % kTcStages]);
          for (uint32_t spin = 0; spin < p.max_spins; ++spin) {
            if (mbar_try_wait(fb, (j / kTcStages) & 1)) break;
            __nanosleep(64);
          }
        }
      }
    }
  } else if (warp >= 9) {
    // ------------------------------------------------------------ MMA issuers: warp 9 -> A block 0, warp 10 -> A block 1
    // The whole warp runs the loop, so that everything the instructions need (descriptors, addresses, parities) is
    // computed once per warp in converged code; one lane issues.  A thread on its own runs one dependent instruction
    // after the other at several cycles each, a wait costs 100-150 cycles even on a finished phase and an MMA or a
    // commit about 50, and the loop is part of the hand-over ring of the accumulators.  So it is kept to the bare
    // sequence: a codebook stage (eight steps) is one trip, its steps are unrolled with constant buffer numbers,
    // parities and descriptor offsets, and a wait that is already over costs a single poll.
    {
      const uint32_t q = (uint32_t)warp - 9u;
      uint64_t a_desc[D::kMmas];
#pragma unroll
      for (int m = 0; m < D::kMmas; ++m)
        a_desc[m] = smem_desc(smem_u32(&sm.a[q][0]), D::kAGroupBytes) + (uint64_t)(D::a_chunk(m) * (128 >> 4));
      uint32_t total = 0;  // steps of this CTA
      for (uint64_t u = blockIdx.x; u < units; u += gridDim.x) {
        uint32_t s_lo, s_hi;
        slice_units(p, (uint32_t)(u % p.n_slices), &s_lo, &s_hi);
        total += s_hi - s_lo;
      }
      const uint64_t b_desc0 = smem_desc(smem_u32(&sm.b[0][0][0]), D::kBGroupBytes);
      const uint32_t full0 = smem_u32(&sm.tmem_full[0][q]), full1 = smem_u32(&sm.tmem_full[1][q]);
      const uint32_t empty0 = smem_u32(&sm.tmem_empty[0][q]), empty1 = smem_u32(&sm.tmem_empty[1][q]);
      const uint32_t d0 = tmem_base + q * 128, d1 = d0 + 256;
      const uint32_t a_ready = smem_u32(&sm.a_ready);
      // a wait whose answer is the same in every lane: one poll by all of them when the phase is already over,
      // otherwise lane 0 polls (bounded) and tells the others
      auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
        if (__all_sync(0xffffffffu, mbar_try_wait(bar, parity))) return true;
        bool ok = true;
        if (lane == 0) ok = mbar_wait(bar, parity, abort_flag, p.status, p.max_spins);
        return __shfl_sync(0xffffffffu, ok, 0);
      };
      bool alive = true;
      uint64_t u = blockIdx.x;
      uint32_t it = 0, unit_i = 0, left = 0;  // steps issued; units begun; steps left in the unit
      uint32_t s = 0, stage_par = 0;          // codebook stage of the trip and the parity of its barrier
      while (it < total && alive) {
        alive = wait_all(smem_u32(&sm.full_bar[s]), stage_par);
        const uint64_t b_s = b_desc0 + (uint64_t)(s * kTcGroupSteps * (kStepBytes >> 4));
#pragma unroll
        for (int sub = 0; sub < kTcGroupSteps; ++sub) {
          if (it < total && alive) {
            if (left == 0) {  // the next unit begins: its A rows must be in place
              uint32_t s_lo, s_hi;
              slice_units(p, (uint32_t)(u % p.n_slices), &s_lo, &s_hi);
              left = s_hi - s_lo;
              u += gridDim.x;
              alive = wait_all(a_ready, unit_i & 1);
              ++unit_i;
            }
            // step 8 g + sub uses buffer sub & 1, for the (4 g + sub / 2)-th time
            if (alive) alive = wait_all((sub & 1) ? empty1 : empty0, ((sub >> 1) & 1) ? 0u : 1u);
            if (alive) {
              tc_fence_after();
              if (lane == 0) {
                // two K chunks per instruction (see TcDim for which chunks of A meet which chunks of B)
#pragma unroll
                for (int m = 0; m < D::kMmas; ++m)
                  umma_f16((sub & 1) ? d1 : d0, a_desc[m],
                           b_s + (uint64_t)(sub * (kStepBytes >> 4) + D::b_chunk(m) * (128 >> 4)), kIdesc, m > 0);
                umma_commit((sub & 1) ? full1 : full0);  // the accumulator is ready
              }
              __syncwarp();
              ++it;
              --left;
            }
          }
        }
        // this warp has read the whole stage (the last stage is not reused)
        if (alive && it < total && lane == 0) umma_commit(smem_u32(&sm.empty_bar[s]));
        __syncwarp();
        s = (s == (uint32_t)kTcStages - 1) ? 0 : s + 1;
        if (s == 0) stage_par ^= 1;
      }
      if (!alive && lane == 0) {
        // wait (bounded) for whatever was issued before tensor memory is released
        umma_commit(smem_u32(&sm.drain_bar[q]));
        for (uint32_t spin = 0; spin < kMaxSpins; ++spin) {  // always the full limit: these MMAs do complete
          if (mbar_try_wait(smem_u32(&sm.drain_bar[q]), 0)) break;
          __nanosleep(64);
        }
      }
    }
  } else {
    // ------------------------------------------------------------ target owners / epilogue
    const float n2max = __uint_as_float(stats->n2max_bits);
    const float cnmax = sqrtf(n2max), hmax = 0.5f * n2max;
    const uint32_t rb = (uint32_t)tid >> 7, r = (uint32_t)tid & 127u;
    unsigned char* a_row = &sm.a[rb][(r >> 3) * D::kAGroupBytes + (r & 7) * 16];
    const uint32_t lane_base = ((uint32_t)(warp & 3) * 32u) << 16;
    uint32_t it = 0;
    bool alive = true;

    for (uint64_t u = blockIdx.x; u < units && alive; u += gridDim.x) {
      const uint32_t tile = (uint32_t)(u / p.n_slices), sl = (uint32_t)(u % p.n_slices);
      uint32_t s_lo, s_hi;
      slice_units(p, sl, &s_lo, &s_hi);
      const uint64_t n = (uint64_t)tile * kTcTile + tid;

      // the target of this thread, its scaling, its A row
      float t[DG];
#pragma unroll
      for (int i = 0; i < DG; ++i) t[i] = 0.0f;
      bool have = false;
      if (n < p.k) {
        const uint32_t j = p.idx[n];
        if (j < p.G) {  // an index out of range is reported by the rescoring kernel
          if (DG == 8)
            form_target(p, j, t);
          else
            form_target16(p, j, t);
          have = true;
        }
      }
      float m = 0.0f, nt2 = 0.0f;
#pragma unroll
      for (int i = 0; i < DG; ++i) {
        m = fmaxf(m, fabsf(t[i]));
        nt2 = fmaf(t[i], t[i], nt2);
      }
      bool in_range = (m < 256.0f) && (nt2 == nt2);  // also false for Inf / NaN
      int e = 0;
      if (in_range && m > 0.0f) {
        e = -ilogbf(m) - 1;
        e = e > 15 ? 15 : e;
      }
      const float sc = in_range ? scalbnf(1.0f, e) : 0.0f;
      {
        __half2 hi[DG / 2], lo[DG / 2];
#pragma unroll
        for (int i = 0; i < DG / 2; ++i) {
          const float x = in_range ? t[2 * i] * sc : 0.0f, y = in_range ? t[2 * i + 1] * sc : 0.0f;  // exact products
          hi[i] = __floats2half2_rn(x, y);
          const float2 back = __half22float2(hi[i]);
          lo[i] = __floats2half2_rn(x - back.x, y - back.y);  // exact differences, rounded once
        }
        const __half2 s2 = __floats2half2_rn(sc, sc);
        const uint32_t sb = *reinterpret_cast<const uint32_t*>(&s2);
        if (DG == 8) {  // [ hi | 2^e | lo | 0 ]
          *reinterpret_cast<uint4*>(a_row) = reinterpret_cast<const uint4*>(hi)[0];
          *reinterpret_cast<uint4*>(a_row + 128) = make_uint4(sb, sb, sb, sb);
          *reinterpret_cast<uint4*>(a_row + 256) = reinterpret_cast<const uint4*>(lo)[0];
          *reinterpret_cast<uint4*>(a_row + 384) = make_uint4(0, 0, 0, 0);
        } else {        // [ hi x 16 | lo x 16 | 2^e | 0 ]
#pragma unroll
          for (int part = 0; part < D::kPart; ++part) {
            *reinterpret_cast<uint4*>(a_row + 128 * part) = reinterpret_cast<const uint4*>(hi)[part];
            *reinterpret_cast<uint4*>(a_row + 128 * (D::kPart + part)) = reinterpret_cast<const uint4*>(lo)[part];
          }
          *reinterpret_cast<uint4*>(a_row + 128 * (2 * D::kPart)) = make_uint4(sb, sb, sb, sb);
          *reinterpret_cast<uint4*>(a_row + 128 * (2 * D::kPart + 1)) = make_uint4(0, 0, 0, 0);
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the MMA
      mbar_arrive(smem_u32(&sm.a_ready));

      // twice the error bound of the fast score, in its own (scaled) units, with a factor 2 to spare.
      // |hi + lo - 2^e t_i| <= 2^-22 |2^e t_i| (2^-25 where lo is subnormal); the norm split is exact to
      // 2^-33 h; products of halves are exact in fp32; the accumulation of at most 32 terms in fp32, rounded
      // or truncated, stays below 2^-19 of the sum of magnitudes 2^e (||t|| ||c|| + h)
      // (48 terms instead of 32 for groups of 16: the factor is doubled there)
      const float margin = sc * (DG == 8 ? 1.52587890625e-5f /* 2^-16 */ : 3.0517578125e-5f /* 2^-15 */) *
                               (sqrtf(nt2) * cnmax + hmax) +
                           4.76837158203125e-7f /* 2^-21 */ * cnmax + 1e-30f;
      float best = kNegInf, thr = kNegInf;

      // Software-pipelined epilogue.  The 128 columns of a step are read as two halves into two register sets, and
      // nothing that has to wait for a result is asked for right after it was requested: the second half is
      // requested before the maxima of the first, the barrier of the next step is tested (without blocking) before
      // those maxima and the answer used after them, and a maximum is compared with the threshold one half later,
      // together with its successor.  A buffer goes back to the MMA warp as soon as both halves are in registers.
      uint32_t v[64], w[64];
      bool pending = false;  // the first half of step `st` is already in flight
      // the list of remembered sub-chunks lives in shared memory, its fill count and the largest evicted maximum
      // in registers: the common case of an event is two stores and no load
      uint32_t list_cnt = 0;
      float evicted_max = kNegInf;
      auto note = [&](float mx, uint32_t sub) {
        if (mx >= thr) {
          const uint32_t slot = list_cnt & (kListLen - 1);
          if (list_cnt >= kListLen) evicted_max = fmaxf(evicted_max, sm.list_max[slot][tid]);
          sm.list_id[slot][tid] = (uint16_t)sub;
          sm.list_max[slot][tid] = mx;
          ++list_cnt;
          best = fmaxf(best, mx);
          thr = best - margin;
        }
      };
      float mx_prev = kNegInf;  // maximum of the previous step's second half, not yet compared
      uint32_t sub_prev = 0;
      for (uint32_t st = s_lo; st < s_hi; ++st, ++it) {
        const uint32_t buf = it & 1;
        const uint32_t taddr = tmem_base + lane_base + buf * 256 + rb * 128;
        if (!pending) {
          // one lane polls (256 threads polling one barrier slow every barrier operation of the CTA
          // down); the warp-wide exchange orders the other lanes after its observation
          const uint32_t fbar = smem_u32(&sm.tmem_full[buf][rb]), fpar = (it >> 1) & 1;
          if (!__all_sync(0xffffffffu, mbar_try_wait(fbar, fpar))) {
            bool ok = true;
            if (lane == 0) ok = mbar_wait(fbar, fpar, abort_flag, p.status, p.max_spins);
            alive = __shfl_sync(0xffffffffu, ok, 0);
            if (!alive) break;
          }
          tc_fence_after();
          tmem_ld64(taddr, v);
        }
        tmem_ld_wait(v);
        tmem_ld64(taddr + 64, w);
        const uint32_t nbuf = (it + 1) & 1;
        uint32_t early = 0;  // is the next step's accumulator complete?  asked now, looked at after the maxima
        if (st + 1 < s_hi)
          early = mbar_test_wait(smem_u32(&sm.tmem_full[nbuf][rb]), ((it + 1) >> 1) & 1);
        const float mv = max64(v);
        tmem_ld_wait(w);
        tc_fence_before();
        mbar_arrive(smem_u32(&sm.tmem_empty[buf][rb]));
        pending = false;
        if (__all_sync(0xffffffffu, early != 0)) {
          tc_fence_after();
          tmem_ld64(tmem_base + lane_base + nbuf * 256 + rb * 128, v);
          pending = true;
        }
        const float mw = max64(w);
        if (fmaxf(mx_prev, mv) >= thr) {
          note(mx_prev, sub_prev);
          note(mv, 2 * st);
        }
        mx_prev = mw;
        sub_prev = 2 * st + 1;
      }
      if (alive) note(mx_prev, sub_prev);

      // leave the candidates of this (tile, slice) for the rescoring kernel (minimum convention: -S)
      if (alive && have) {
        CandRecord rec;
        rec.pad = 0;
        uint32_t cnt_out = 0;
#pragma unroll
        for (int q = 0; q < kListLen; ++q) rec.sub[q] = 0;
        if (in_range) {
          const float limit = best - margin;
          const uint32_t cnt = list_cnt;
#pragma unroll
          for (int q = 0; q < kListLen; ++q)
            if ((uint32_t)q < cnt && sm.list_max[q][tid] >= limit) rec.sub[cnt_out++] = sm.list_id[q][tid];
          rec.best = -best;
          rec.cnt = (cnt > (uint32_t)kListLen && evicted_max >= limit) ? kCandOverflow : (uint16_t)cnt_out;
        } else {
          rec.best = kNegInf;  // passes every limit: the whole slice is rescored exactly
          rec.cnt = kCandOverflow;
        }
        *reinterpret_cast<uint4*>(&p.rec[((size_t)tile * p.n_slices + sl) * kTcTile + tid]) =
            *reinterpret_cast<const uint4*>(&rec);
        atomicMin(&p.gbest[n], ord(rec.best));
        if (sl == 0) p.margin[n] = in_range ? margin : 0.0f;
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace

namespace {

template <int DG>
cudaError_t launch_tc(const pvt_layer& L, const EncM1Params& p, const EncodeM1TcLayout& lay, char* base, TcStats* stats,
                      cudaStream_t stream) {
  timing_begin(kKernEncodeAux, stream);
  const uint32_t n_cw = lay.n_steps * kTcStepCw;
  tc_prep_kernel<DG><<<(n_cw + 255) / 256, 256, 0, stream>>>(
      reinterpret_cast<const uint4*>(L.codebooks), p.K, lay.n_steps,
      reinterpret_cast<unsigned char*>(base + lay.bimg_off), stats, reinterpret_cast<uint32_t*>(base + lay.exc_off));
  count_launches(1);
  timing_end(kKernEncodeAux, stream);
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  const size_t smem = sizeof(TcSmem<DG>);
  if ((err = cudaFuncSetAttribute(encode_m1_tc_kernel<DG>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) !=
      cudaSuccess)
    return err;
  timing_begin(kKernEncodeMain, stream);
  encode_m1_tc_kernel<DG><<<lay.n_ctas, kTcThreads, smem, stream>>>(
      p, reinterpret_cast<const unsigned char*>(base + lay.bimg_off), stats);
  timing_end(kKernEncodeMain, stream);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_encode_m1_tc(const pvt_layer& L, uint64_t G, const uint32_t* idx, uint64_t k, float* err_out,
                                void* ws, int sm_count, cudaStream_t stream) {
  const EncodeM1TcLayout lay = encode_m1_tc_layout((uint32_t)L.codebook_size, k, sm_count, L.group_dim);
  char* base = static_cast<char*>(ws);
  TcStats* stats = reinterpret_cast<TcStats*>(base + lay.stats_off);
  EncM1Params p;
  p.W = L.W;
  p.g = L.g;
  p.scale = L.scale;
  p.idx = idx;
  p.k = k;
  p.G = G;
  p.gpr = (uint32_t)(L.cols / L.group_dim);
  p.dg = (uint32_t)L.group_dim;
  p.eta = L.eta;
  p.cbx = nullptr;
  p.n2max_bits = &stats->n2max_bits;
  p.K = (uint32_t)L.codebook_size;
  p.n_tiles = lay.n_tiles;
  p.n_slices = lay.n_slices;
  p.tile = kTcTile;
  p.n_units = lay.n_steps;
  p.unit_cw = kTcStepCw;
  p.sub_cw = kTcSubCw;
  p.exc_count = &stats->exc_count;
  p.exc_list = reinterpret_cast<const uint32_t*>(base + lay.exc_off);
  p.gbest = reinterpret_cast<uint32_t*>(base + lay.gbest_off);
  p.margin = reinterpret_cast<float*>(base + lay.margin_off);
  p.rec = reinterpret_cast<CandRecord*>(base + lay.rec_off);
  p.book = L.codebooks;
  p.codes = L.codes;
  p.code_u16 = L.code_dtype == PVT_U16;
  p.err_out = err_out;
  p.status = reinterpret_cast<uint32_t*>(base);
  const WaitTestHook hook = wait_test_hook();
  p.max_spins = hook.max_spins;
  p.withhold_copy = hook.withhold_copy;

  cudaError_t err = cudaMemsetAsync(stats, 0, sizeof(TcStats), stream);
  if (err != cudaSuccess) return err;
  if ((err = cudaMemsetAsync(p.gbest, 0xff, sizeof(uint32_t) * k, stream)) != cudaSuccess) return err;
  err = L.group_dim == 16 ? launch_tc<16>(L, p, lay, base, stats, stream) : launch_tc<8>(L, p, lay, base, stats, stream);
  if (err != cudaSuccess) return err;
  return launch_rescore_m1(p, true, stream);
}

}  // namespace pvt
