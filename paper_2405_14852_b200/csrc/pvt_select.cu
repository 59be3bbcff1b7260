// Subspace choice of the V step (the top-tau selection of Algorithm 2; Section 3.4 ranks by
// update size, separately for every weight matrix): squared update norm per weight group,
// then an exact top-k by radix select on the binary32 bit patterns, ties at the
// threshold resolved towards the lowest group index, result in ascending order.
//
// Passes (all on one stream, no host round trip, no inter-block waiting):
//   1. norm_hist:   persistent grid; read g once (32 B per group), write the key of
//                   every group, histogram key bits [30:20]
//   2. refine_mid:  read the keys; those inside the threshold bucket are
//                   histogrammed on bits [19:9] and copied to a compact candidate
//                   list (usually a few per cent of the groups)
//   3. refine_low:  histogram bits [8:0] of the candidates that match both digits
//   4. tile_count:  per tile of 4096 groups: how many keys > threshold, == threshold
//   5. scatter:     ordered compaction: position = (#greater before) +
//                   min(#equal before, number of ties to take)
// In passes 1-4 the block that finishes last (atomic ticket, no spinning) turns
// the histogram into the next threshold digit, or the tile counts into offsets.
#include "pvt_internal.h"

namespace pvt {

SelectLayout select_layout(uint64_t G) {
  SelectLayout s;
  s.ntiles = (uint32_t)((G + kSelTile - 1) / kSelTile);
  // candidates: a quarter of the groups is far more than a threshold bucket of real gradients holds; when
  // it is not enough (many equal norms) the low pass reads the keys instead
  uint64_t cap = G / 4;
  if (cap < 65536) cap = 65536;
  if (cap > G) cap = G;
  s.cand_cap = (uint32_t)cap;
  s.hist_off = kWsHeaderBytes;
  s.keys_off = align_up(s.hist_off + sizeof(uint32_t) * (kSelBins0 + kSelBins1 + kSelBins2), kWsAlign);
  s.tiles_off = align_up(s.keys_off + sizeof(uint32_t) * G, kWsAlign);
  s.cand_off = align_up(s.tiles_off + sizeof(uint32_t) * 2 * (size_t)s.ntiles, kWsAlign);
  s.bytes = align_up(s.cand_off + sizeof(uint32_t) * (size_t)s.cand_cap, kWsAlign);
  return s;
}

namespace {

// Keys: n_j = ||eta * g_j||^2 in binary32: u = eta*g_i rounded once, acc = fma(u, u, acc)
// in index order from 0.  Non-negative, so the bit pattern orders like the value.

// Block-wide: true in every thread of the block that took the last ticket.
__device__ __forceinline__ bool last_block_done(uint32_t* counter) {
  __shared__ bool is_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint32_t ticket = atomicAdd(counter, 1u);
    is_last = (ticket == gridDim.x - 1);
  }
  __syncthreads();
  if (is_last) __threadfence();
  return is_last;
}

// Inclusive scan of one value per thread over a block of kSelThreads threads.
__device__ __forceinline__ uint64_t block_inclusive_scan(uint64_t v, uint64_t* sh /*[kSelThreads/32]*/) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint64_t n = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += n;
  }
  __syncthreads();
  if (lane == 31) sh[warp] = v;
  __syncthreads();
  uint64_t base = 0;
  for (int w = 0; w < warp; ++w) base += sh[w];
  return v + base;
}

// Walk a histogram from its top bin downwards and find the bin that holds the
// k_left-th largest key.  Exactly one thread of the block finds it and writes
// *digit and *k_new (= how many keys must still be taken from inside that bin).
template <int NBINS>
__device__ void find_digit(const uint32_t* hist, uint64_t k_left, uint32_t* digit, uint64_t* k_new,
                           uint64_t* sh_scan) {
  constexpr int PER = NBINS / kSelThreads;
  // thread t owns the bins [hi - PER + 1, hi], hi descending with t
  const int hi = NBINS - 1 - threadIdx.x * PER;
  uint32_t c[PER];
  uint64_t mine = 0;
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    c[i] = __ldcg(hist + hi - i);
    mine += c[i];
  }
  const uint64_t incl = block_inclusive_scan(mine, sh_scan);
  uint64_t above = incl - mine;  // keys in bins above this thread's bins
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    if (above < k_left && k_left <= above + c[i]) {
      *digit = (uint32_t)(hi - i);
      *k_new = k_left - above;
    }
    above += c[i];
  }
}

constexpr int kNormPer = 8;                              // 16-byte loads per thread and iteration of the norm pass

// LP adjacent lanes share a group (LP = group size / 4: 2 or 4), lane q of them holding elements 4q..4q+3,
// so a warp reads 512 contiguous bytes per load instruction.  The sum is a single chain in index order:
// lane 0 runs its four steps from 0 and hands the partial sum to lane 1, which runs the next four, and so
// on; every lane computes every round (the work is free, the pass is bound by memory), the value is
// kept only where it is the group's own partial sum.
__device__ __forceinline__ float norm_chain(float acc, const float4& a, float eta) {
  float u;
  u = __fmul_rn(eta, a.x); acc = __fmaf_rn(u, u, acc);
  u = __fmul_rn(eta, a.y); acc = __fmaf_rn(u, u, acc);
  u = __fmul_rn(eta, a.z); acc = __fmaf_rn(u, u, acc);
  u = __fmul_rn(eta, a.w); acc = __fmaf_rn(u, u, acc);
  return acc;
}

// ---- random subspace rules (appendix on small-scale experiments: subspaces drawn uniformly at random, or at
// random in proportion to the size of the gradient entries) --------------------------------------------------
// Every group gets the first output word of Philox-4x32 with 10 rounds (Salmon et al., SC 2011) at counter
// (j mod 2^32, j div 2^32, 0, 0) under the key (seed mod 2^32, seed div 2^32).
__device__ __forceinline__ uint32_t philox_first_word(uint64_t j, uint64_t seed) {
  uint32_t c0 = (uint32_t)j, c1 = (uint32_t)(j >> 32), c2 = 0u, c3 = 0u;
  uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint32_t h0 = __umulhi(0xD2511F53u, c0), l0 = 0xD2511F53u * c0;
    const uint32_t h1 = __umulhi(0xCD9E8D57u, c2), l1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = h1 ^ c1 ^ k0, n2 = h0 ^ c3 ^ k1;
    c0 = n0; c1 = l1; c2 = n2; c3 = l0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return c0;
}

// E = -ln((r + 1/2) 2^-32) by a fixed sequence of binary64 operations (each rounded once, none contracted):
// r + 1/2 = m 2^e, m in [1, 2), m halved and e raised when m > sqrt 2; z = (m - 1)/(m + 1);
// p = 1 + z^2/3 + ... + z^20/21 by Horner's rule, one fused operation per coefficient; E = fma(32 - e, ln 2, -(2z p)).
__device__ __forceinline__ double neglog_u32(uint32_t r) {
  int e = r ? 31 - __clz((int)r) : -1;
  // (r + 1/2) 2^-e, exact: the significand of r + 1/2 with the exponent field set to that of 1.0
  const double x = __dadd_rn((double)r, 0.5);
  double m = __longlong_as_double((__double_as_longlong(x) & 0x000fffffffffffffll) | 0x3ff0000000000000ll);
  if (m > 1.4142135623730951) {
    m = __dmul_rn(m, 0.5);
    e = e + 1;
  }
  const double z = __ddiv_rn(__dadd_rn(m, -1.0), __dadd_rn(m, 1.0)), z2 = __dmul_rn(z, z);
  double p = 1.0 / 21.0;
#pragma unroll
  for (int d = 19; d >= 1; d -= 2) p = __fma_rn(p, z2, 1.0 / (double)d);
  const double lnm = __dmul_rn(__dmul_rn(2.0, z), p);
  return __fma_rn((double)(32 - e), 0.6931471805599453, -lnm);
}

// What the first pass computes per group (everything after the keys is the same top-k):
//   kKeyNorm          key = squared update norm (the greedy rule of the V step)
//   kKeyNormBuffer    the same, and the straight-through buffer takes the step: buffer = fma(-eta, g, buffer)
//   kKeyUniform       key = the top 24 bits of the group's random word, as a binary32 number
//   kKeyProportional  key = (float)(norm / E), E the exponential clock of the group's random word
enum KeyMode { kKeyNorm = 0, kKeyNormBuffer = 1, kKeyUniform = 2, kKeyProportional = 3 };

template <int LP, int MODE>
__global__ void __launch_bounds__(kSelThreads) norm_hist_kernel(const float* __restrict__ g, uint64_t G, float eta,
                                                                 uint64_t k, uint32_t* __restrict__ keys,
                                                                 uint32_t* __restrict__ hist0, SelectState* st,
                                                                 float* __restrict__ buffer, uint64_t seed) {
  pdl_trigger();
  pdl_wait();
  constexpr int kTile = kSelThreads * kNormPer / LP;  // groups per block and iteration
  __shared__ uint32_t sh_hist[kSelBins0];
  __shared__ uint64_t sh_scan[kSelThreads / 32];
  for (int b = threadIdx.x; b < kSelBins0; b += kSelThreads) sh_hist[b] = 0;
  __syncthreads();
  const float4* g4 = reinterpret_cast<const float4*>(g);
  float4* buf4 = reinterpret_cast<float4*>(buffer);
  const uint64_t F = (uint64_t)LP * G;  // 16-byte pieces
  const uint32_t n_tiles = (uint32_t)((G + kTile - 1) / kTile);
  const int q = threadIdx.x & (LP - 1);  // position of this lane within its group
  for (uint32_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const uint64_t f0 = (uint64_t)tile * (LP * kTile) + threadIdx.x;
    float4 a[kNormPer];
#pragma unroll
    for (int i = 0; i < kNormPer; ++i) {  // all loads of the iteration first
      const uint64_t f = f0 + (uint64_t)i * kSelThreads;
      a[i] = (MODE != kKeyUniform && f < F) ? __ldcs(g4 + f) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (MODE == kKeyNormBuffer) {  // the straight-through buffer takes the step of every weight (Appendix E)
      float4 b[kNormPer];
#pragma unroll
      for (int i = 0; i < kNormPer; ++i) {
        const uint64_t f = f0 + (uint64_t)i * kSelThreads;
        b[i] = f < F ? __ldcs(buf4 + f) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
      const float neg_eta = -eta;
#pragma unroll
      for (int i = 0; i < kNormPer; ++i) {
        const uint64_t f = f0 + (uint64_t)i * kSelThreads;
        if (f < F)
          __stcs(buf4 + f, make_float4(__fmaf_rn(neg_eta, a[i].x, b[i].x), __fmaf_rn(neg_eta, a[i].y, b[i].y),
                                       __fmaf_rn(neg_eta, a[i].z, b[i].z), __fmaf_rn(neg_eta, a[i].w, b[i].w)));
      }
    }
#pragma unroll
    for (int i = 0; i < kNormPer; ++i) {
      const uint64_t f = f0 + (uint64_t)i * kSelThreads;
      float acc = norm_chain(0.0f, a[i], eta);  // valid on lane 0 of the group
#pragma unroll
      for (int r = 1; r < LP; ++r) {
        const float in = __shfl_up_sync(0xffffffffu, acc, 1);  // lane r: the sum over elements 0..4r-1
        const float next = norm_chain(in, a[i], eta);
        acc = q >= r ? next : acc;
      }
      if (q == LP - 1 && f < F) {
        uint32_t key = __float_as_uint(acc);
        if (MODE == kKeyUniform) key = __float_as_uint((float)(philox_first_word(f / LP, seed) >> 8));
        if (MODE == kKeyProportional)
          key = acc > 0.0f ? __float_as_uint(__double2float_rn(
                                 __ddiv_rn((double)acc, neglog_u32(philox_first_word(f / LP, seed)))))
                           : 0u;
        keys[f / LP] = key;
        atomicAdd(&sh_hist[key >> 20], 1u);
      }
    }
  }
  __syncthreads();
  for (int b = threadIdx.x; b < kSelBins0; b += kSelThreads)
    if (sh_hist[b]) atomicAdd(&hist0[b], sh_hist[b]);
  if (last_block_done(&st->done[0])) find_digit<kSelBins0>(hist0, k, &st->digit0, &st->k_left, sh_scan);
}

// Keys whose bits [30:20] equal digit0: histogram of bits [19:9], and a compact copy
// (order irrelevant) for the last refinement.  Bucket members are first collected in
// shared memory; a block reserves room in the global list with one atomic per flush.
constexpr int kMidStage = 2048;  // bucket members a block collects before it flushes

__global__ void __launch_bounds__(kSelThreads) refine_mid_kernel(const uint32_t* __restrict__ keys, uint64_t G,
                                                                  uint32_t* __restrict__ hist1,
                                                                  uint32_t* __restrict__ cand, uint32_t cand_cap,
                                                                  SelectState* st) {
  pdl_trigger();
  pdl_wait();
  __shared__ uint32_t sh_hist[kSelBins1];
  __shared__ uint64_t sh_scan[kSelThreads / 32];
  __shared__ uint32_t sh_stage[kMidStage + 8 * kSelThreads];  // room for one more iteration after the check
  __shared__ uint32_t sh_n, sh_base;
  for (int b = threadIdx.x; b < kSelBins1; b += kSelThreads) sh_hist[b] = 0;
  if (threadIdx.x == 0) sh_n = 0;
  __syncthreads();
  const uint32_t prefix = st->digit0;
  const uint64_t n_quads = (G + 3) / 4;
  const uint64_t stride = (uint64_t)gridDim.x * kSelThreads;

  auto flush = [&]() {  // called by the whole block
    __syncthreads();
    const uint32_t n = sh_n;
    if (threadIdx.x == 0 && n) sh_base = atomicAdd(&st->cand_count, n);
    __syncthreads();
    const uint32_t base = sh_base;
    for (uint32_t i = threadIdx.x; i < n; i += kSelThreads)
      if (base + i < cand_cap) cand[base + i] = sh_stage[i];
    __syncthreads();
    if (threadIdx.x == 0) sh_n = 0;
    __syncthreads();
  };

  for (uint64_t q0 = (uint64_t)blockIdx.x * kSelThreads; q0 < n_quads; q0 += 2 * stride) {
    // two independent 16-byte loads per thread and iteration
    uint32_t key[8];
    uint32_t have[2] = {0, 0};
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint64_t q = q0 + (uint64_t)h * stride + threadIdx.x;
#pragma unroll
      for (int i = 0; i < 4; ++i) key[4 * h + i] = 0;
      if (q < n_quads) {
        if (4 * q + 4 <= G) {
          const uint4 v = *reinterpret_cast<const uint4*>(keys + 4 * q);
          key[4 * h] = v.x; key[4 * h + 1] = v.y; key[4 * h + 2] = v.z; key[4 * h + 3] = v.w;
          have[h] = 4;
        } else {
          have[h] = (uint32_t)(G - 4 * q);
          for (uint32_t i = 0; i < have[h]; ++i) key[4 * h + i] = keys[4 * q + i];
        }
      }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if ((uint32_t)i < have[h] && (key[4 * h + i] >> 20) == prefix) {
          atomicAdd(&sh_hist[(key[4 * h + i] >> 9) & 0x7ffu], 1u);
          sh_stage[atomicAdd(&sh_n, 1u)] = key[4 * h + i];
        }
      }
    }
    __syncthreads();
    const uint32_t collected = sh_n;  // the same value in every thread
    __syncthreads();                  // nobody adds to it again before everybody has read it
    if (collected >= (uint32_t)kMidStage) flush();
  }
  flush();
  for (int b = threadIdx.x; b < kSelBins1; b += kSelThreads)
    if (sh_hist[b]) atomicAdd(&hist1[b], sh_hist[b]);
  if (last_block_done(&st->done[1])) {
    const uint64_t k_left = st->k_left;
    __syncthreads();
    find_digit<kSelBins1>(hist1, k_left, &st->digit1, &st->k_left, sh_scan);
  }
}

// Bits [8:0] of the candidates that match (digit0, digit1); reads the candidate list, or
// all keys if the list did not hold every bucket member.
__global__ void __launch_bounds__(kSelThreads) refine_low_kernel(const uint32_t* __restrict__ keys, uint64_t G,
                                                                  const uint32_t* __restrict__ cand,
                                                                  uint32_t cand_cap, uint32_t* __restrict__ hist2,
                                                                  SelectState* st) {
  pdl_trigger();
  pdl_wait();
  __shared__ uint32_t sh_hist[kSelBins2];
  __shared__ uint64_t sh_scan[kSelThreads / 32];
  for (int b = threadIdx.x; b < kSelBins2; b += kSelThreads) sh_hist[b] = 0;
  __syncthreads();
  const uint32_t prefix = (st->digit0 << 11) | st->digit1;
  const uint32_t n_cand = st->cand_count;
  const bool listed = n_cand <= cand_cap;
  const uint32_t* src = listed ? cand : keys;
  const uint64_t n = listed ? (uint64_t)n_cand : G;
  for (uint64_t i = (uint64_t)blockIdx.x * kSelThreads + threadIdx.x; i < n; i += (uint64_t)gridDim.x * kSelThreads) {
    const uint32_t key = src[i];
    if ((key >> 9) == prefix) atomicAdd(&sh_hist[key & 0x1ffu], 1u);
  }
  __syncthreads();
  for (int b = threadIdx.x; b < kSelBins2; b += kSelThreads)
    if (sh_hist[b]) atomicAdd(&hist2[b], sh_hist[b]);
  if (last_block_done(&st->done[2])) {
    const uint64_t k_left = st->k_left;
    __shared__ uint32_t d2;
    __shared__ uint64_t kn;
    __syncthreads();
    find_digit<kSelBins2>(hist2, k_left, &d2, &kn, sh_scan);
    __syncthreads();
    if (threadIdx.x == 0) {
      st->threshold = (st->digit0 << 20) | (st->digit1 << 9) | d2;
      st->need_eq = (uint32_t)kn;
    }
  }
}

__global__ void __launch_bounds__(kSelThreads) tile_count_kernel(const uint32_t* __restrict__ keys, uint64_t G,
                                                                  uint32_t* __restrict__ tiles, uint32_t ntiles,
                                                                  uint64_t k, SelectState* st, uint32_t* status) {
  pdl_trigger();
  pdl_wait();
  __shared__ uint32_t sh_gt, sh_eq;
  __shared__ uint64_t sh_scan[kSelThreads / 32];
  if (threadIdx.x == 0) sh_gt = sh_eq = 0;
  __syncthreads();
  const uint32_t T = st->threshold;
  const uint64_t j0 = (uint64_t)blockIdx.x * kSelTile;
  constexpr int QUADS = kSelTile / (4 * kSelThreads);  // 16-byte loads per thread, all issued before use
  uint32_t gt = 0, eq = 0;
  if (j0 + kSelTile <= G) {
    uint4 v[QUADS];
#pragma unroll
    for (int i = 0; i < QUADS; ++i)
      v[i] = *reinterpret_cast<const uint4*>(keys + j0 + 4 * ((uint64_t)i * kSelThreads + threadIdx.x));
#pragma unroll
    for (int i = 0; i < QUADS; ++i) {
      gt += (v[i].x > T) + (v[i].y > T) + (v[i].z > T) + (v[i].w > T);
      eq += (v[i].x == T) + (v[i].y == T) + (v[i].z == T) + (v[i].w == T);
    }
  } else {
    for (uint64_t j = j0 + threadIdx.x; j < G; j += kSelThreads) {
      const uint32_t key = keys[j];
      gt += key > T;
      eq += key == T;
    }
  }
  gt = __reduce_add_sync(0xffffffffu, gt);
  eq = __reduce_add_sync(0xffffffffu, eq);
  if ((threadIdx.x & 31) == 0) {
    if (gt) atomicAdd(&sh_gt, gt);
    if (eq) atomicAdd(&sh_eq, eq);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    tiles[2 * blockIdx.x] = sh_gt;
    tiles[2 * blockIdx.x + 1] = sh_eq;
  }
  if (last_block_done(&st->done[3])) {
    // exclusive scan of the tile counts, in place; consecutive tiles per thread
    const uint32_t per = (ntiles + kSelThreads - 1) / kSelThreads;
    const uint32_t lo = min(threadIdx.x * per, ntiles), hi = min(lo + per, ntiles);
    uint64_t sg = 0, se = 0;
    for (uint32_t t = lo; t < hi; ++t) {
      sg += __ldcg(tiles + 2 * t);
      se += __ldcg(tiles + 2 * t + 1);
    }
    const uint64_t ig = block_inclusive_scan(sg, sh_scan);
    __syncthreads();
    const uint64_t ie = block_inclusive_scan(se, sh_scan);
    uint64_t rg = ig - sg, re = ie - se;
    for (uint32_t t = lo; t < hi; ++t) {
      const uint32_t cg = __ldcg(tiles + 2 * t), ce = __ldcg(tiles + 2 * t + 1);
      tiles[2 * t] = (uint32_t)rg;
      tiles[2 * t + 1] = (uint32_t)re;
      rg += cg;
      re += ce;
    }
    if (threadIdx.x == kSelThreads - 1) {
      // all greater keys plus the ties taken must be exactly k
      const uint64_t taken_eq = ie < st->need_eq ? ie : st->need_eq;
      if (ig + taken_eq != k) atomicOr(status, PVT_DEV_INTERNAL);
    }
  }
}

__global__ void __launch_bounds__(kSelThreads) scatter_kernel(const uint32_t* __restrict__ keys, uint64_t G,
                                                               const uint32_t* __restrict__ tiles,
                                                               const SelectState* st, uint64_t k,
                                                               uint32_t* __restrict__ idx_out) {
  pdl_trigger();
  pdl_wait();
  __shared__ uint64_t sh_scan[kSelThreads / 32];
  const uint32_t T = st->threshold, need_eq = st->need_eq;
  constexpr int PER = kSelTile / kSelThreads;  // consecutive groups per thread: keeps index order
  const uint64_t jt = (uint64_t)blockIdx.x * kSelTile + (uint64_t)threadIdx.x * PER;
  uint32_t key[PER];
  if (jt + PER <= G) {
    const uint4* p = reinterpret_cast<const uint4*>(keys + jt);
#pragma unroll
    for (int i = 0; i < PER / 4; ++i) {
      const uint4 v = p[i];
      key[4 * i] = v.x; key[4 * i + 1] = v.y; key[4 * i + 2] = v.z; key[4 * i + 3] = v.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < PER; ++i) key[i] = (jt + i < G) ? keys[jt + i] : 0u;
  }
  uint32_t gt = 0, eq = 0;
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    const bool in = jt + i < G;
    gt += in && key[i] > T;
    eq += in && key[i] == T;
  }
  // one scan for both counts: each fits 16 bits inside a tile of 4096
  const uint64_t packed = (uint64_t)gt | ((uint64_t)eq << 32);
  const uint64_t incl = block_inclusive_scan(packed, sh_scan);
  uint64_t GT = (uint64_t)tiles[2 * blockIdx.x] + (uint32_t)(incl - packed);
  uint64_t EQ = (uint64_t)tiles[2 * blockIdx.x + 1] + (uint32_t)((incl - packed) >> 32);
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    if (jt + i < G) {
      const bool is_gt = key[i] > T, is_eq = key[i] == T;
      if (is_gt || (is_eq && EQ < need_eq)) {
        const uint64_t pos = GT + (EQ < need_eq ? EQ : need_eq);
        if (pos < k) idx_out[pos] = (uint32_t)(jt + i);
      }
      GT += is_gt;
      EQ += is_eq;
    }
  }
}

__global__ void iota_kernel(uint32_t* idx_out, uint64_t k) {
  const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < k) idx_out[i] = (uint32_t)i;
}

}  // namespace

namespace {

template <int LP, int MODE>
cudaError_t launch_norm(const pvt_layer& L, uint64_t G, uint64_t k, uint32_t* keys, uint32_t* hist0, SelectState* st,
                        float* buffer, uint64_t seed, int sm_count, cudaStream_t stream) {
  int per_sm = 0;
  cudaError_t err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, norm_hist_kernel<LP, MODE>, kSelThreads, 0);
  if (err != cudaSuccess) return err;
  const uint64_t tile = (uint64_t)kSelThreads * kNormPer / LP;
  const uint64_t tiles = (G + tile - 1) / tile;
  const uint64_t resident = (uint64_t)sm_count * (uint64_t)(per_sm > 0 ? per_sm : 1);  // a persistent grid
  norm_hist_kernel<LP, MODE><<<(unsigned)(tiles < resident ? tiles : resident), kSelThreads, 0, stream>>>(
      L.g, G, L.eta, k, keys, hist0, st, buffer, seed);
  return cudaGetLastError();
}

template <int LP>
cudaError_t launch_norm_mode(int mode, const pvt_layer& L, uint64_t G, uint64_t k, uint32_t* keys, uint32_t* hist0,
                             SelectState* st, float* buffer, uint64_t seed, int sm_count, cudaStream_t stream) {
  switch (mode) {
    case kKeyNormBuffer: return launch_norm<LP, kKeyNormBuffer>(L, G, k, keys, hist0, st, buffer, seed, sm_count, stream);
    case kKeyUniform: return launch_norm<LP, kKeyUniform>(L, G, k, keys, hist0, st, buffer, seed, sm_count, stream);
    case kKeyProportional:
      return launch_norm<LP, kKeyProportional>(L, G, k, keys, hist0, st, buffer, seed, sm_count, stream);
    default: return launch_norm<LP, kKeyNorm>(L, G, k, keys, hist0, st, buffer, seed, sm_count, stream);
  }
}

}  // namespace

cudaError_t launch_select(const pvt_layer& L, uint64_t G, uint64_t k, uint32_t* idx_out, void* ws, int sm_count,
                          cudaStream_t stream) {
  return launch_select_keyed(L, G, k, idx_out, ws, sm_count, stream, kKeyNorm, nullptr, 0);
}

cudaError_t launch_select_keyed(const pvt_layer& L, uint64_t G, uint64_t k, uint32_t* idx_out, void* ws, int sm_count,
                                cudaStream_t stream, int key_mode, float* buffer, uint64_t seed) {
  timing_begin(kKernSelect, stream);
  cudaError_t err = cudaSuccess;
  if (k == G && key_mode != kKeyNormBuffer) {  // every group is taken: the ascending index list itself
    iota_kernel<<<(unsigned)((k + 255) / 256), 256, 0, stream>>>(idx_out, k);
    err = cudaGetLastError();
    count_launches(1);
    timing_end(kKernSelect, stream);
    return err;
  }
  const SelectLayout lay = select_layout(G);
  char* base = static_cast<char*>(ws);
  uint32_t* status = reinterpret_cast<uint32_t*>(base);
  SelectState* st = reinterpret_cast<SelectState*>(base + kSelStateOffset);
  uint32_t* hist0 = reinterpret_cast<uint32_t*>(base + lay.hist_off);
  uint32_t* hist1 = hist0 + kSelBins0;
  uint32_t* hist2 = hist1 + kSelBins1;
  uint32_t* keys = reinterpret_cast<uint32_t*>(base + lay.keys_off);
  uint32_t* tiles = reinterpret_cast<uint32_t*>(base + lay.tiles_off);
  // selection state (header, from byte 64) and the three histograms are adjacent: one clear
  static_assert(kSelStateOffset + sizeof(SelectState) <= kWsHeaderBytes, "selection state must fit the header");
  if ((err = cudaMemsetAsync(st, 0, (kWsHeaderBytes - kSelStateOffset) +
                                        sizeof(uint32_t) * (kSelBins0 + kSelBins1 + kSelBins2), stream)) !=
      cudaSuccess)
    return err;
  uint32_t* cand = reinterpret_cast<uint32_t*>(base + lay.cand_off);
  // persistent grids: exactly the blocks that are resident at once
  int mid_per_sm = 0;
  if ((err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&mid_per_sm, refine_mid_kernel, kSelThreads, 0)) !=
      cudaSuccess)
    return err;
  const uint64_t quad_blocks = ((G + 3) / 4 + 2 * kSelThreads - 1) / (2 * kSelThreads);
  const uint64_t mid_res = (uint64_t)sm_count * (uint64_t)(mid_per_sm > 0 ? mid_per_sm : 1);
  const unsigned mid_grid = (unsigned)(quad_blocks < mid_res ? quad_blocks : mid_res);
  err = L.group_dim == 16 ? launch_norm_mode<4>(key_mode, L, G, k, keys, hist0, st, buffer, seed, sm_count, stream)
                          : launch_norm_mode<2>(key_mode, L, G, k, keys, hist0, st, buffer, seed, sm_count, stream);
  if (err != cudaSuccess) return err;
  err = launch_dependent(refine_mid_kernel, mid_grid, kSelThreads, 0, stream, keys, G, hist1, cand, lay.cand_cap, st);
  if (err != cudaSuccess) return err;
  const unsigned low_grid = (unsigned)(lay.cand_cap / 8192 < (uint32_t)sm_count ? lay.cand_cap / 8192 + 1 : sm_count);
  err = launch_dependent(refine_low_kernel, low_grid, kSelThreads, 0, stream, keys, G, cand, lay.cand_cap, hist2, st);
  if (err != cudaSuccess) return err;
  err = launch_dependent(tile_count_kernel, lay.ntiles, kSelThreads, 0, stream, keys, G, tiles, lay.ntiles, k, st, status);
  if (err != cudaSuccess) return err;
  err = launch_dependent(scatter_kernel, lay.ntiles, kSelThreads, 0, stream, keys, G, tiles, st, k, idx_out);
  if (err == cudaSuccess) err = cudaGetLastError();
  count_launches(5);
  timing_end(kKernSelect, stream);
  return err;
}

}  // namespace pvt
