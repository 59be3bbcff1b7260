// Exhaustive nearest-codeword search of the V step for one codebook (Appendix C /
// Appendix J: all codewords of the codebook are tried; Appendix D: the score
// ||c||^2 - 2 <t, c>; Eq. 8 for the target t = (W - eta g) / s).
//
// Two kernels.
//
// Search.  Targets are cut into tiles of 256*TT groups, the codebook into slices
// of whole 256-codeword chunks; the (tile, slice) units are dealt round-robin to
// one persistent CTA per SM.  Per unit:
//   1. every compute thread gathers TT targets (32 B of W and of g each), forms t
//      in binary32 and keeps -t in registers, duplicated into f32x2 pairs;
//   2. a producer warp streams the pre-expanded codebook (pairs of codewords
//      interleaved, half squared norms appended) chunk by chunk into a 4-stage
//      shared-memory ring with 1-D bulk tensor-memory-accelerator copies that
//      complete on mbarriers;
//   3. the compute warps read one codeword pair per iteration (broadcast loads)
//      and evaluate score = ||c||^2/2 - <t, c> for both codewords and all TT
//      targets with packed fma.rn.f32x2, folding the two scores into a running
//      minimum with one three-input min: 8 FMAs and half a min per pair
//      evaluation, no distance matrix, no index tracking in the hot loop;
//   4. every 32 codewords the running minimum of that sub-chunk is compared with
//      the best so far; sub-chunks within a rounding-error margin of the best are
//      remembered (4 most recent per target);
//   5. at the end of the unit each thread writes, per target, the remembered
//      sub-chunks that are still within the margin of the slice minimum, and folds
//      the slice minimum into a per-target global minimum (atomic).
// Rescoring.  One warp per target: every remembered sub-chunk of every slice whose
// minimum lies within the margin of the global minimum is revisited, the binary64
// distance sum (t_i-c_i)^2 (index order) of each of its codewords is evaluated
// from the caller's codebook, and the argmin of (distance, code) is written.
// The margin bounds twice the rounding error of the fast score, so the codeword
// that is nearest in exact arithmetic is always among those rescored.
#include <cuda_fp16.h>

#include "pvt_encode_m1.cuh"

namespace pvt {

EncodeM1Layout encode_m1_layout(uint32_t K, uint64_t k, int sm_count, int tt) {
  EncodeM1Layout e;
  e.n_chunks = (K + kChunkCodewords - 1) / kChunkCodewords;
  e.tile = (uint32_t)(kEncThreads * tt);
  e.n_tiles = (uint32_t)((k + e.tile - 1) / e.tile);
  // slices: the fewest that keep the last round of units over the SMs nearly full
  uint32_t best_s = 1;
  double best_eff = 0.0;
  const uint32_t s_max = e.n_chunks < (uint32_t)kMaxSlices ? e.n_chunks : (uint32_t)kMaxSlices;
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
  e.cbx_off = kWsHeaderBytes;
  e.n2max_off = align_up(e.cbx_off + (size_t)e.n_chunks * kChunkBytes, kWsAlign);
  e.gbest_off = e.n2max_off + kWsAlign;
  e.margin_off = align_up(e.gbest_off + sizeof(uint32_t) * k, kWsAlign);
  e.rec_off = align_up(e.margin_off + sizeof(float) * k, kWsAlign);
  e.bytes = align_up(e.rec_off + (size_t)e.n_tiles * e.n_slices * e.tile * sizeof(CandRecord), kWsAlign);
  return e;
}

int encode_m1_targets_per_thread(uint64_t k, int sm_count) {
  // 8 targets per thread amortise the shared-memory reads best, but tiles of 2048
  // targets only pay off when there are many tiles per SM
  return k >= (uint64_t)sm_count * 2048ull * 4ull ? 8 : 4;
}

using namespace m1;

namespace {

constexpr float kPadHalfNorm = 3.0e38f;  // half norm of padding codewords: never near a minimum

// ---- codebook expansion ------------------------------------------------------
// chunk block (kChunkBytes): 128 pairs * 16 floats, pair p holds
// (c[2p][0], c[2p+1][0], c[2p][1], c[2p+1][1], ...), then 128 * 2 half norms.
template <bool CB_F16>
__global__ void expand_codebook_kernel(const void* __restrict__ book, uint32_t K, uint32_t n_chunks,
                                       float* __restrict__ cbx, uint32_t* __restrict__ n2max_bits) {
  const uint32_t kappa = blockIdx.x * blockDim.x + threadIdx.x;
  float n2 = 0.0f;
  if (kappa < n_chunks * kChunkCodewords) {
    float c[8];
    if (kappa < K) {
      if (CB_F16) {
        const uint4 raw = reinterpret_cast<const uint4*>(book)[kappa];
        const __half2* h = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f = __half22float2(h[i]);
          c[2 * i] = f.x;
          c[2 * i + 1] = f.y;
        }
      } else {
        const float4* p = reinterpret_cast<const float4*>(book) + 2 * (size_t)kappa;
        const float4 a = p[0], b = p[1];
        c[0] = a.x; c[1] = a.y; c[2] = a.z; c[3] = a.w;
        c[4] = b.x; c[5] = b.y; c[6] = b.z; c[7] = b.w;
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) n2 = __fmaf_rn(c[i], c[i], n2);
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) c[i] = 0.0f;
    }
    const uint32_t chunk = kappa / kChunkCodewords, w = kappa % kChunkCodewords;
    float* blk = cbx + (size_t)chunk * (kChunkBytes / 4);
    const uint32_t pr = w >> 1, half = w & 1;
#pragma unroll
    for (int i = 0; i < 8; ++i) blk[pr * 16 + 2 * i + half] = c[i];
    blk[kChunkCodewords * 8 + pr * 2 + half] = kappa < K ? __fmul_rn(0.5f, n2) : kPadHalfNorm;
  }
  // max ||c||^2 over the codebook (non-negative floats order like their bit patterns)
  uint32_t bits = __float_as_uint(n2);
  bits = __reduce_max_sync(0xffffffffu, bits);
  if ((threadIdx.x & 31) == 0 && bits > __ldcg(n2max_bits)) atomicMax(n2max_bits, bits);
}

__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ float min3(float a, float b, float c) {
  float d;
  asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  return (uint64_t)__float_as_uint(lo) | ((uint64_t)__float_as_uint(hi) << 32);
}
// ---- shared-memory layout of the search kernel -----------------------------------
template <int TT>
struct EncSmem {
  static constexpr int TILE = kEncThreads * TT;
  alignas(128) unsigned char stage[kEncStages][kChunkBytes];
  alignas(8) uint64_t full_bar[kEncStages];
  uint64_t empty_bar[kEncStages];
  float evicted_min[TILE];            // smallest sub-chunk minimum that fell out of the list
  float list_min[kListLen][TILE];
  uint16_t list_id[kListLen][TILE];
  uint16_t list_cnt[TILE];
  uint32_t abort_flag;
};

template <int TT>
__global__ void __launch_bounds__(kEncThreads + 32, 1) encode_m1_kernel(const EncM1Params p) {
  using Smem = EncSmem<TT>;
  constexpr int TILE = Smem::TILE;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  volatile uint32_t* abort_flag = &sm.abort_flag;

  if (tid == 0) {
    sm.abort_flag = 0;
    for (int s = 0; s < kEncStages; ++s) {
      mbar_init(smem_u32(&sm.full_bar[s]), 1);
      mbar_init(smem_u32(&sm.empty_bar[s]), kEncThreads / 32);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  const uint64_t units = (uint64_t)p.n_tiles * p.n_slices;

  if (warp == kEncThreads / 32) {
    // ------------------------------------------------------------ producer warp
    if (lane == 0) {
      uint32_t it = 0;
      bool alive = true;
      for (uint64_t u = blockIdx.x; u < units && alive; u += gridDim.x) {
        const uint32_t sl = (uint32_t)(u % p.n_slices);
        uint32_t c_lo, c_hi;
        slice_units(p, sl, &c_lo, &c_hi);
        for (uint32_t c = c_lo; c < c_hi && alive; ++c, ++it) {
          const uint32_t s = it % kEncStages;
          if (it >= kEncStages)
            alive = mbar_wait(smem_u32(&sm.empty_bar[s]), ((it / kEncStages) - 1) & 1, abort_flag, p.status, p.max_spins);
          if (!alive) break;
          if (it == p.withhold_copy) continue;  // test hook: this chunk never arrives, its consumers' wait runs out
          const uint32_t fb = smem_u32(&sm.full_bar[s]);
          mbar_expect_tx(fb, kChunkBytes);
          bulk_g2s(smem_u32(&sm.stage[s][0]), reinterpret_cast<const char*>(p.cbx) + (size_t)c * kChunkBytes,
                   kChunkBytes, fb);
        }
      }
      if (!alive) {
        // drain: let every copy that was issued land before the CTA may exit
        for (uint32_t back = 1; back <= kEncStages && back <= it; ++back) {
          const uint32_t j = it - back;
          if (j == p.withhold_copy) continue;  // never issued
          const uint32_t fb = smem_u32(&sm.full_bar[j % kEncStages]);
          for (uint32_t spin = 0; spin < p.max_spins; ++spin) {
            if (mbar_try_wait(fb, (j / kEncStages) & 1)) break;
            __nanosleep(64);
          }
        }
      }
    }
    return;
  }

  // -------------------------------------------------------------- compute warps
  const float n2max = __uint_as_float(*p.n2max_bits);
  uint32_t it = 0;

  for (uint64_t u = blockIdx.x; u < units; u += gridDim.x) {
    const uint32_t tile = (uint32_t)(u / p.n_slices);
    const uint32_t sl = (uint32_t)(u % p.n_slices);
    uint32_t c_lo, c_hi;
    slice_units(p, sl, &c_lo, &c_hi);

    // 1. gather targets, form t, set up tracking
    uint64_t nt[TT][8];  // (-t_i, -t_i)
    float thr[TT], best[TT], margin[TT];
#pragma unroll
    for (int tt = 0; tt < TT; ++tt) {
      const int s = tt * kEncThreads + tid;
      const uint64_t n = (uint64_t)tile * TILE + s;
      float t[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) t[i] = 0.0f;
      if (n < p.k) {
        const uint32_t j = p.idx[n];
        if (j < p.G) form_target(p, j, t);  // an index out of range is reported by the rescoring kernel
      }
      float nt2 = 0.0f;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        nt2 = fmaf(t[i], t[i], nt2);
        nt[tt][i] = pack2(-t[i], -t[i]);
      }
      // twice the rounding-error bound of the fast score, with a factor 2 to spare:
      // |score_fl - score| <= 16.1 u (||c||^2/2 + ||t|| ||c||), u = 2^-24
      margin[tt] = 3.8146973e-6f /* 2^-18 */ * (0.5f * n2max + sqrtf(nt2 * n2max)) + 1e-30f;
      best[tt] = __int_as_float(0x7f800000);
      thr[tt] = best[tt];
      sm.list_cnt[s] = 0;
      sm.evicted_min[s] = __int_as_float(0x7f800000);
    }

    // 2.-4. stream the codebook chunks of this slice
    for (uint32_t c = c_lo; c < c_hi; ++c, ++it) {
      const uint32_t st = it % kEncStages;
      mbar_wait(smem_u32(&sm.full_bar[st]), (it / kEncStages) & 1, abort_flag, p.status, p.max_spins);
      const unsigned char* stage = &sm.stage[st][0];
#pragma unroll 1
      for (int sub = 0; sub < kChunkCodewords / kSubCodewords; ++sub) {
        float cmin[TT];
#pragma unroll
        for (int tt = 0; tt < TT; ++tt) cmin[tt] = __int_as_float(0x7f800000);
        const ulonglong2* vals = reinterpret_cast<const ulonglong2*>(stage) + sub * (kSubCodewords / 2) * 4;
        const uint64_t* norms =
            reinterpret_cast<const uint64_t*>(stage + kChunkCodewords * 32) + sub * (kSubCodewords / 2);
#pragma unroll 4
        for (int pr = 0; pr < kSubCodewords / 2; ++pr) {
          const ulonglong2 q0 = vals[4 * pr], q1 = vals[4 * pr + 1], q2 = vals[4 * pr + 2], q3 = vals[4 * pr + 3];
          const uint64_t h = norms[pr];
#pragma unroll
          for (int tt = 0; tt < TT; ++tt) {
            uint64_t acc = h;
            acc = fma2(nt[tt][0], q0.x, acc);
            acc = fma2(nt[tt][1], q0.y, acc);
            acc = fma2(nt[tt][2], q1.x, acc);
            acc = fma2(nt[tt][3], q1.y, acc);
            acc = fma2(nt[tt][4], q2.x, acc);
            acc = fma2(nt[tt][5], q2.y, acc);
            acc = fma2(nt[tt][6], q3.x, acc);
            acc = fma2(nt[tt][7], q3.y, acc);
            cmin[tt] = min3(cmin[tt], __uint_as_float((uint32_t)acc), __uint_as_float((uint32_t)(acc >> 32)));
          }
        }
        const uint32_t sub_id = c * (kChunkCodewords / kSubCodewords) + sub;
#pragma unroll
        for (int tt = 0; tt < TT; ++tt) {
          if (cmin[tt] <= thr[tt]) {
            const int s = tt * kEncThreads + tid;
            const uint32_t cnt = sm.list_cnt[s];
            const uint32_t slot = cnt & (kListLen - 1);
            if (cnt >= kListLen) sm.evicted_min[s] = fminf(sm.evicted_min[s], sm.list_min[slot][s]);
            sm.list_id[slot][s] = (uint16_t)sub_id;
            sm.list_min[slot][s] = cmin[tt];
            sm.list_cnt[s] = (uint16_t)(cnt + 1);
            best[tt] = fminf(best[tt], cmin[tt]);
            thr[tt] = best[tt] + margin[tt];
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&sm.empty_bar[st]));
    }

    // 5. leave the candidates of this (tile, slice) for the rescoring kernel
    if (*abort_flag == 0) {
#pragma unroll
      for (int tt = 0; tt < TT; ++tt) {
        const int s = tt * kEncThreads + tid;
        const uint64_t n = (uint64_t)tile * TILE + s;
        if (n >= p.k) continue;
        const float limit = best[tt] + margin[tt];
        const uint32_t cnt = sm.list_cnt[s];
        CandRecord r;
        r.best = best[tt];
        r.pad = 0;
        uint32_t m = 0;
#pragma unroll
        for (int v = 0; v < kListLen; ++v) {
          r.sub[v] = 0;
          if ((uint32_t)v < cnt && sm.list_min[v][s] <= limit) r.sub[m++] = sm.list_id[v][s];
        }
        r.cnt = (cnt > (uint32_t)kListLen && sm.evicted_min[s] <= limit) ? kCandOverflow : (uint16_t)m;
        *reinterpret_cast<uint4*>(&p.rec[((size_t)tile * p.n_slices + sl) * TILE + s]) =
            *reinterpret_cast<const uint4*>(&r);
        atomicMin(&p.gbest[n], ord(best[tt]));
        if (sl == 0) p.margin[n] = margin[tt];
      }
    }
  }
}

// ---- rescoring --------------------------------------------------------------------
template <bool CB_F16, int DG>
__device__ __forceinline__ void load_codeword(const void* book, uint32_t kappa, float* c) {
  if (CB_F16) {
#pragma unroll
    for (int part = 0; part < DG / 8; ++part) {
      const uint4 raw = __ldg(reinterpret_cast<const uint4*>(book) + (size_t)kappa * (DG / 8) + part);
      const __half2* h = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(h[i]);
        c[8 * part + 2 * i] = f.x;
        c[8 * part + 2 * i + 1] = f.y;
      }
    }
  } else {
    const float4* q = reinterpret_cast<const float4*>(book) + (size_t)kappa * (DG / 4);
#pragma unroll
    for (int part = 0; part < DG / 4; ++part) {
      const float4 a = __ldg(q + part);
      c[4 * part] = a.x; c[4 * part + 1] = a.y; c[4 * part + 2] = a.z; c[4 * part + 3] = a.w;
    }
  }
}

// Eight lanes per target, four targets per warp: the kernel is a chain of dependent memory round trips
// ((index, global minimum, margin, records) -> (W, g, scale) -> codewords), so what counts is how many targets
// are in flight per warp, not how fast one of them is evaluated.
constexpr int kRsLanes = 8;
constexpr int kRsPerWarp = 32 / kRsLanes;
constexpr int kRsPerBlock = 8 * kRsPerWarp;  // 256 threads
static_assert(kMaxSlices <= 2 * kRsLanes, "two records per lane must cover every slice");

template <bool CB_F16, int DG>
__global__ void __launch_bounds__(256) rescore_m1_kernel(const EncM1Params p) {
  constexpr uint32_t kFull = 0xffffffffu;
  const uint32_t sub_cw = p.sub_cw;
  const int lane = threadIdx.x & 31, grp = lane / kRsLanes, l = lane % kRsLanes;
  const int gshift = grp * kRsLanes;
  const uint64_t n = ((uint64_t)blockIdx.x * 8 + (threadIdx.x >> 5)) * kRsPerWarp + grp;
  bool active = n < p.k;
  uint32_t j = 0;
  float limit = 0.0f;
  uint4 raw0 = make_uint4(0x7f800000u, 0, 0, 0), raw1 = raw0;  // best = +inf: never within the limit
  if (active) {
    const uint32_t tile = (uint32_t)(n / p.tile), s = (uint32_t)(n % p.tile);
    j = __ldg(p.idx + n);
    limit = unord(p.gbest[n]) + p.margin[n];
    const uint4* rec = reinterpret_cast<const uint4*>(p.rec);
    if ((uint32_t)l < p.n_slices) raw0 = __ldg(&rec[((size_t)tile * p.n_slices + l) * p.tile + s]);
    if ((uint32_t)l + kRsLanes < p.n_slices)
      raw1 = __ldg(&rec[((size_t)tile * p.n_slices + l + kRsLanes) * p.tile + s]);
    if (j >= p.G) {
      if (l == 0) atomicOr(p.status, PVT_DEV_BAD_INDEX);
      active = false;
    }
  }
  float t[DG];
#pragma unroll
  for (int i = 0; i < DG; ++i) t[i] = 0.0f;
  if (active) {
    if (DG == 8)
      form_target(p, j, t);
    else
      form_target16(p, j, t);
  }
  const uint32_t subs_per_unit = p.unit_cw / sub_cw;
  double best_d = __longlong_as_double(0x7ff0000000000000ll);
  uint32_t best_code = 0xffffffffu;

  auto score = [&](uint32_t kappa) {
    float c[DG];
    load_codeword<CB_F16, DG>(p.book, kappa, c);
    double d = 0.0;
#pragma unroll
    for (int i = 0; i < DG; ++i) {
      const double e = __dsub_rn((double)t[i], (double)c[i]);
      d = __dadd_rn(d, __dmul_rn(e, e));
    }
    if (d < best_d || (d == best_d && kappa < best_code)) {
      best_d = d;
      best_code = kappa;
    }
  };
  auto visit = [&](uint32_t sub) {
    for (uint32_t w = l; w < sub_cw; w += kRsLanes) {
      const uint32_t kappa = sub * sub_cw + w;
      if (kappa < p.K) score(kappa);
    }
  };

  // slices whose minimum lies within the margin of the global minimum: bit s of `live`, the same in the
  // eight lanes of a target.  The loop runs while any target of the warp has a slice left, so that the
  // shuffles are executed by the whole warp.
  const uint32_t in0 = __ballot_sync(kFull, active && __uint_as_float(raw0.x) <= limit);
  const uint32_t in1 = __ballot_sync(kFull, active && __uint_as_float(raw1.x) <= limit);
  uint32_t live = ((in0 >> gshift) & 0xffu) | (((in1 >> gshift) & 0xffu) << kRsLanes);
  while (__any_sync(kFull, live != 0)) {
    const bool has = live != 0;
    const int sl = has ? __ffs(live) - 1 : 0;
    live &= live - 1;
    const int src = gshift + (sl & (kRsLanes - 1));
    const bool upper = sl >= kRsLanes;
    const uint32_t y0 = __shfl_sync(kFull, raw0.y, src), y1 = __shfl_sync(kFull, raw1.y, src);
    const uint32_t z0 = __shfl_sync(kFull, raw0.z, src), z1 = __shfl_sync(kFull, raw1.z, src);
    const uint32_t w0 = __shfl_sync(kFull, raw0.w, src), w1 = __shfl_sync(kFull, raw1.w, src);
    if (!has) continue;
    const uint32_t s01 = upper ? y1 : y0, s23 = upper ? z1 : z0;
    const uint32_t cnt = (upper ? w1 : w0) & 0xffffu;
    if (cnt == kCandOverflow) {
      uint32_t u_lo, u_hi;
      slice_units(p, (uint32_t)sl, &u_lo, &u_hi);
      for (uint32_t sub = u_lo * subs_per_unit; sub < u_hi * subs_per_unit; ++sub) visit(sub);
    } else {
      if (cnt > 0) visit(s01 & 0xffffu);
      if (cnt > 1) visit(s01 >> 16);
      if (cnt > 2) visit(s23 & 0xffffu);
      if (cnt > 3) visit(s23 >> 16);
    }
  }
  if (p.exc_count && active) {  // codewords whose fast score is not trustworthy: always evaluated
    const uint32_t n_exc = __ldg(p.exc_count);
    for (uint32_t e = l; e < n_exc && e < p.K; e += kRsLanes) {
      const uint32_t kappa = __ldg(p.exc_list + e);
      if (kappa < p.K) score(kappa);
    }
  }
  // lexicographic minimum of (distance, code) over the eight lanes of the target; distances are >= 0 so their
  // bits order like u64
  const uint64_t bits = (uint64_t)__double_as_longlong(best_d);
  uint32_t hi = (uint32_t)(bits >> 32), lo = (uint32_t)bits, code = best_code;
#pragma unroll
  for (int off = kRsLanes / 2; off > 0; off >>= 1) {
    const uint32_t ohi = __shfl_xor_sync(kFull, hi, off), olo = __shfl_xor_sync(kFull, lo, off);
    const uint32_t ocode = __shfl_xor_sync(kFull, code, off);
    if (ohi < hi || (ohi == hi && (olo < lo || (olo == lo && ocode < code)))) {
      hi = ohi;
      lo = olo;
      code = ocode;
    }
  }
  if (l == 0 && active) {
    if (code < p.K) {
      if (p.code_u16)
        reinterpret_cast<uint16_t*>(p.codes)[j] = (uint16_t)code;
      else
        reinterpret_cast<uint8_t*>(p.codes)[j] = (uint8_t)code;
      if (p.err_out) p.err_out[n] = (float)__longlong_as_double((long long)(((uint64_t)hi << 32) | lo));
    } else {
      atomicOr(p.status, PVT_DEV_INTERNAL);  // no candidate survived: the search did not complete
    }
  }
}

template <int TT>
cudaError_t launch_tt(const EncM1Params& p, uint32_t n_ctas, cudaStream_t stream) {
  const size_t smem = sizeof(EncSmem<TT>);
  cudaError_t err = cudaFuncSetAttribute(encode_m1_kernel<TT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (err != cudaSuccess) return err;
  timing_begin(kKernEncodeMain, stream);
  encode_m1_kernel<TT><<<n_ctas, kEncThreads + 32, smem, stream>>>(p);
  timing_end(kKernEncodeMain, stream);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_encode_m1(const pvt_layer& L, uint64_t G, const uint32_t* idx, uint64_t k, float* err_out,
                             void* ws, int sm_count, cudaStream_t stream) {
  const int tt = encode_m1_targets_per_thread(k, sm_count);
  const EncodeM1Layout lay = encode_m1_layout((uint32_t)L.codebook_size, k, sm_count, tt);
  char* base = static_cast<char*>(ws);
  EncM1Params p;
  p.W = L.W;
  p.g = L.g;
  p.scale = L.scale;
  p.idx = idx;
  p.k = k;
  p.G = G;
  p.gpr = (uint32_t)(L.cols / kGroupDim);
  p.dg = kGroupDim;
  p.eta = L.eta;
  p.cbx = reinterpret_cast<const float*>(base + lay.cbx_off);
  p.n2max_bits = reinterpret_cast<const uint32_t*>(base + lay.n2max_off);
  p.n_units = lay.n_chunks;
  p.unit_cw = kChunkCodewords;
  p.sub_cw = kSubCodewords;
  p.exc_count = nullptr;
  p.exc_list = nullptr;
  p.K = (uint32_t)L.codebook_size;
  p.n_tiles = lay.n_tiles;
  p.n_slices = lay.n_slices;
  p.tile = lay.tile;
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

  cudaError_t err = cudaMemsetAsync(base + lay.n2max_off, 0, sizeof(uint32_t), stream);
  if (err != cudaSuccess) return err;
  if ((err = cudaMemsetAsync(p.gbest, 0xff, sizeof(uint32_t) * k, stream)) != cudaSuccess) return err;
  timing_begin(kKernEncodeAux, stream);
  const uint32_t n_cw = lay.n_chunks * kChunkCodewords;
  const bool f16 = L.codebook_dtype == PVT_F16;
  if (f16)
    expand_codebook_kernel<true><<<(n_cw + 255) / 256, 256, 0, stream>>>(
        L.codebooks, p.K, lay.n_chunks, const_cast<float*>(p.cbx), const_cast<uint32_t*>(p.n2max_bits));
  else
    expand_codebook_kernel<false><<<(n_cw + 255) / 256, 256, 0, stream>>>(
        L.codebooks, p.K, lay.n_chunks, const_cast<float*>(p.cbx), const_cast<uint32_t*>(p.n2max_bits));
  count_launches(1);
  timing_end(kKernEncodeAux, stream);
  if ((err = cudaGetLastError()) != cudaSuccess) return err;
  err = tt == 8 ? launch_tt<8>(p, lay.n_ctas, stream) : launch_tt<4>(p, lay.n_ctas, stream);
  if (err != cudaSuccess) return err;
  return launch_rescore_m1(p, f16, stream);
}

cudaError_t launch_rescore_m1(const EncM1Params& p, bool codebook_f16, cudaStream_t stream) {
  timing_begin(kKernEncodeRescore, stream);
  const unsigned blocks = (unsigned)((p.k + kRsPerBlock - 1) / kRsPerBlock);
  if (p.dg == 16) {  // groups of 16 weights come from the tensor engine only: fp16 codebooks
    rescore_m1_kernel<true, 16><<<blocks, 256, 0, stream>>>(p);
  } else if (codebook_f16) {
    rescore_m1_kernel<true, 8><<<blocks, 256, 0, stream>>>(p);
  } else {
    rescore_m1_kernel<false, 8><<<blocks, 256, 0, stream>>>(p);
  }
  count_launches(1);
  timing_end(kKernEncodeRescore, stream);
  return cudaGetLastError();
}

}  // namespace pvt
