// Pieces shared by the two M = 1 search kernels (FP32 pipe and tensor cores) and
// the rescoring kernel that follows either: parameters, the binary32 target, the
// order-preserving float <-> u32 map, mbarrier / bulk-copy PTX wrappers.
#pragma once

#include <cuda_fp16.h>

#include "pvt_internal.h"

namespace pvt {
namespace m1 {

constexpr uint32_t kMaxSpins = 1u << 22;     // polls after which a wait on an on-chip barrier gives up
constexpr uint32_t kNoWithhold = 0xffffffffu;

// Test hook for the give-up path of the waits (host side, process-wide): the poll limit the search kernels
// run with, and the number of one codebook copy that the producer leaves out so that a wait really runs out.
struct WaitTestHook {
  uint32_t max_spins;      // kMaxSpins unless a test lowered it
  uint32_t withhold_copy;  // kNoWithhold, or the per-CTA sequence number of the copy that is never issued
};
WaitTestHook wait_test_hook();
void set_wait_test_hook(uint32_t max_spins, uint32_t withhold_copy);

struct EncM1Params {
  const float* W;
  const float* g;
  const float* scale;
  const uint32_t* idx;
  uint64_t k, G;
  uint32_t gpr;
  uint32_t dg;  // weights per group: 8, or 16 (tensor engine and rescoring only)
  float eta;
  const float* cbx;
  const uint32_t* n2max_bits;
  uint32_t K, n_tiles, n_slices, tile;
  uint32_t n_units, unit_cw;  // the codebook is cut into n_units units of unit_cw codewords; a slice is a run of whole units
  uint32_t sub_cw;            // codewords per remembered sub-chunk (a multiple of 32 that divides unit_cw)
  const uint32_t* exc_count;  // codewords the fast score cannot represent: always rescored (may be null)
  const uint32_t* exc_list;
  uint32_t* gbest;
  float* margin;
  CandRecord* rec;
  const void* book;  // the caller's codebook [K][dg]
  void* codes;
  int code_u16;
  float* err_out;
  uint32_t* status;
  uint32_t max_spins;      // poll limit of every wait on an on-chip barrier
  uint32_t withhold_copy;  // kNoWithhold; otherwise the producer skips its copy of this sequence number (test hook)
};

// order-preserving map binary32 -> u32 (and back)
__device__ __forceinline__ uint32_t ord(float f) {
  const uint32_t b = __float_as_uint(f);
  return b ^ ((b >> 31) ? 0xffffffffu : 0x80000000u);
}
__device__ __forceinline__ float unord(uint32_t o) {
  return __uint_as_float(o ^ ((o >> 31) ? 0x80000000u : 0xffffffffu));
}

// t = (W - eta g) / s of group j in binary32: one fma, one division per element
__device__ __forceinline__ void form_target(const EncM1Params& p, uint32_t j, float* t) {
  const float4* W4 = reinterpret_cast<const float4*>(p.W);
  const float4* g4 = reinterpret_cast<const float4*>(p.g);
  const float4 w0 = __ldg(W4 + 2 * (size_t)j), w1 = __ldg(W4 + 2 * (size_t)j + 1);
  const float4 g0 = __ldg(g4 + 2 * (size_t)j), g1 = __ldg(g4 + 2 * (size_t)j + 1);
  const float sc = __ldg(p.scale + j / p.gpr);
  const float neg_eta = -p.eta;
  t[0] = __fdiv_rn(__fmaf_rn(neg_eta, g0.x, w0.x), sc);
  t[1] = __fdiv_rn(__fmaf_rn(neg_eta, g0.y, w0.y), sc);
  t[2] = __fdiv_rn(__fmaf_rn(neg_eta, g0.z, w0.z), sc);
  t[3] = __fdiv_rn(__fmaf_rn(neg_eta, g0.w, w0.w), sc);
  t[4] = __fdiv_rn(__fmaf_rn(neg_eta, g1.x, w1.x), sc);
  t[5] = __fdiv_rn(__fmaf_rn(neg_eta, g1.y, w1.y), sc);
  t[6] = __fdiv_rn(__fmaf_rn(neg_eta, g1.z, w1.z), sc);
  t[7] = __fdiv_rn(__fmaf_rn(neg_eta, g1.w, w1.w), sc);
}

// the same for a group of 16 weights
__device__ __forceinline__ void form_target16(const EncM1Params& p, uint32_t j, float* t) {
  const float4* W4 = reinterpret_cast<const float4*>(p.W) + 4 * (size_t)j;
  const float4* g4 = reinterpret_cast<const float4*>(p.g) + 4 * (size_t)j;
  const float sc = __ldg(p.scale + j / p.gpr);
  const float neg_eta = -p.eta;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float4 w = __ldg(W4 + q), gg = __ldg(g4 + q);
    t[4 * q + 0] = __fdiv_rn(__fmaf_rn(neg_eta, gg.x, w.x), sc);
    t[4 * q + 1] = __fdiv_rn(__fmaf_rn(neg_eta, gg.y, w.y), sc);
    t[4 * q + 2] = __fdiv_rn(__fmaf_rn(neg_eta, gg.z, w.z), sc);
    t[4 * q + 3] = __fdiv_rn(__fmaf_rn(neg_eta, gg.w, w.w), sc);
  }
}

// ---- PTX helpers ---------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// 1-D bulk copy global -> shared through the tensor memory accelerator; completes
// `bytes` on the mbarrier.  Both addresses 16-byte aligned, bytes % 16 == 0.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
// Bounded wait.  Gives up after max_spins polls (or as soon as another thread gave
// up), flags the CTA as aborted and reports through the status word.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t* status, uint32_t max_spins) {
  for (uint32_t spin = 0; spin < max_spins; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (spin > 4096) __nanosleep(64);  // try_wait itself suspends the thread for a short while
  }
  *abort_flag = 1;
  atomicOr(status, PVT_DEV_WAIT_EXPIRED);
  return false;
}


// units [lo, hi) of slice sl
__device__ __forceinline__ void slice_units(const EncM1Params& p, uint32_t sl, uint32_t* lo, uint32_t* hi) {
  *lo = (uint32_t)((uint64_t)sl * p.n_units / p.n_slices);
  *hi = (uint32_t)((uint64_t)(sl + 1) * p.n_units / p.n_slices);
}

}  // namespace m1

// exact rescoring + code write after either search kernel (defined with the FP32 search)
cudaError_t launch_rescore_m1(const m1::EncM1Params& p, bool codebook_f16, cudaStream_t stream);

}  // namespace pvt
