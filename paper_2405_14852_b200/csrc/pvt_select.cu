// Subspace choice of the V step (Algorithm 2 "arg top tau"; Section 3.4 "largest
// update norm within each weight matrix"): squared update norm per weight group,
// then an exact top-k by radix select on the binary32 bit patterns, ties at the
// threshold resolved towards the lowest group index, result in ascending order.
//
// Passes (all on one stream, no host round trip, no inter-block waiting):
//   1. norm_hist:   read g once (32 B per group), write the key of every group,
//                   histogram key bits [30:20]
//   2. hist_mid:    histogram bits [19:9] of the keys inside the threshold bucket
//   3. hist_low:    histogram bits [8:0] of the keys that match both digits
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
  s.hist_off = kWsHeaderBytes;
  s.keys_off = align_up(s.hist_off + sizeof(uint32_t) * (kSelBins0 + kSelBins1 + kSelBins2), kWsAlign);
  s.tiles_off = align_up(s.keys_off + sizeof(uint32_t) * G, kWsAlign);
  s.bytes = align_up(s.tiles_off + sizeof(uint32_t) * 2 * (size_t)s.ntiles, kWsAlign);
  return s;
}

namespace {

// n_j = ||eta * g_j||^2 in binary32: u = eta*g_i rounded once, acc = fma(u, u, acc)
// in index order from 0.  Non-negative, so the bit pattern orders like the value.
__device__ __forceinline__ uint32_t group_key(const float4 a, const float4 b, float eta) {
  float acc = 0.0f, u;
  u = __fmul_rn(eta, a.x); acc = __fmaf_rn(u, u, acc);
  u = __fmul_rn(eta, a.y); acc = __fmaf_rn(u, u, acc);
  u = __fmul_rn(eta, a.z); acc = __fmaf_rn(u, u, acc);
  u = __fmul_rn(eta, a.w); acc = __fmaf_rn(u, u, acc);
  u = __fmul_rn(eta, b.x); acc = __fmaf_rn(u, u, acc);
  u = __fmul_rn(eta, b.y); acc = __fmaf_rn(u, u, acc);
  u = __fmul_rn(eta, b.z); acc = __fmaf_rn(u, u, acc);
  u = __fmul_rn(eta, b.w); acc = __fmaf_rn(u, u, acc);
  return __float_as_uint(acc);
}

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

__device__ __forceinline__ void hist_add_matched(uint32_t* sh_hist, uint32_t bin, bool valid) {
  // one shared-memory atomic per distinct bin of the warp: synthetic gradients put
  // most keys of a warp into a handful of bins
  const uint32_t b = valid ? bin : 0xffffffffu;
  const uint32_t peers = __match_any_sync(0xffffffffu, b);
  if (valid && (threadIdx.x & 31) == (uint32_t)(__ffs(peers) - 1)) atomicAdd(&sh_hist[bin], (uint32_t)__popc(peers));
}

__global__ void __launch_bounds__(kSelThreads) norm_hist_kernel(const float* __restrict__ g, uint64_t G, float eta,
                                                                 uint64_t k, uint32_t* __restrict__ keys,
                                                                 uint32_t* __restrict__ hist0, SelectState* st) {
  __shared__ uint32_t sh_hist[kSelBins0];
  __shared__ uint64_t sh_scan[kSelThreads / 32];
  for (int b = threadIdx.x; b < kSelBins0; b += kSelThreads) sh_hist[b] = 0;
  __syncthreads();
  const uint64_t j0 = (uint64_t)blockIdx.x * kSelTile;
  const float4* g4 = reinterpret_cast<const float4*>(g);
  constexpr int PER = kSelTile / kSelThreads;
#pragma unroll 4
  for (int i = 0; i < PER; ++i) {
    const uint64_t j = j0 + (uint64_t)i * kSelThreads + threadIdx.x;
    const bool valid = j < G;
    uint32_t key = 0;
    if (valid) {
      const float4 a = __ldcs(g4 + 2 * j), b = __ldcs(g4 + 2 * j + 1);
      key = group_key(a, b, eta);
      keys[j] = key;
    }
    hist_add_matched(sh_hist, key >> 20, valid);
  }
  __syncthreads();
  for (int b = threadIdx.x; b < kSelBins0; b += kSelThreads)
    if (sh_hist[b]) atomicAdd(&hist0[b], sh_hist[b]);
  if (last_block_done(&st->done[0])) find_digit<kSelBins0>(hist0, k, &st->digit0, &st->k_left, sh_scan);
}

// PASS 1: bins = key bits [19:9] of keys whose bits [30:20] equal digit0.
// PASS 2: bins = key bits [8:0] of keys whose bits [30:9] equal (digit0, digit1).
template <int PASS>
__global__ void __launch_bounds__(kSelThreads) hist_refine_kernel(const uint32_t* __restrict__ keys, uint64_t G,
                                                                   uint32_t* __restrict__ hist, SelectState* st) {
  constexpr int NBINS = PASS == 1 ? kSelBins1 : kSelBins2;
  __shared__ uint32_t sh_hist[NBINS];
  __shared__ uint64_t sh_scan[kSelThreads / 32];
  for (int b = threadIdx.x; b < NBINS; b += kSelThreads) sh_hist[b] = 0;
  __syncthreads();
  const uint32_t prefix = PASS == 1 ? st->digit0 : ((st->digit0 << 11) | st->digit1);
  const uint64_t j0 = (uint64_t)blockIdx.x * kSelTile;
  constexpr int PER = kSelTile / kSelThreads;
#pragma unroll 4
  for (int i = 0; i < PER; ++i) {
    const uint64_t j = j0 + (uint64_t)i * kSelThreads + threadIdx.x;
    if (j < G) {
      const uint32_t key = keys[j];
      if (PASS == 1) {
        if ((key >> 20) == prefix) atomicAdd(&sh_hist[(key >> 9) & 0x7ffu], 1u);
      } else {
        if ((key >> 9) == prefix) atomicAdd(&sh_hist[key & 0x1ffu], 1u);
      }
    }
  }
  __syncthreads();
  for (int b = threadIdx.x; b < NBINS; b += kSelThreads)
    if (sh_hist[b]) atomicAdd(&hist[b], sh_hist[b]);
  if (last_block_done(&st->done[PASS])) {
    const uint64_t k_left = st->k_left;
    __syncthreads();
    if (PASS == 1) {
      find_digit<NBINS>(hist, k_left, &st->digit1, &st->k_left, sh_scan);
    } else {
      __shared__ uint32_t d2;
      __shared__ uint64_t kn;
      find_digit<NBINS>(hist, k_left, &d2, &kn, sh_scan);
      __syncthreads();
      if (threadIdx.x == 0) {
        st->threshold = (st->digit0 << 20) | (st->digit1 << 9) | d2;
        st->need_eq = (uint32_t)kn;
      }
    }
  }
}

__global__ void __launch_bounds__(kSelThreads) tile_count_kernel(const uint32_t* __restrict__ keys, uint64_t G,
                                                                  uint32_t* __restrict__ tiles, uint32_t ntiles,
                                                                  uint64_t k, SelectState* st, uint32_t* status) {
  __shared__ uint32_t sh_gt, sh_eq;
  __shared__ uint64_t sh_scan[kSelThreads / 32];
  if (threadIdx.x == 0) sh_gt = sh_eq = 0;
  __syncthreads();
  const uint32_t T = st->threshold;
  const uint64_t j0 = (uint64_t)blockIdx.x * kSelTile;
  constexpr int PER = kSelTile / kSelThreads;
  uint32_t gt = 0, eq = 0;
#pragma unroll 4
  for (int i = 0; i < PER; ++i) {
    const uint64_t j = j0 + (uint64_t)i * kSelThreads + threadIdx.x;
    if (j < G) {
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

cudaError_t launch_select(const pvt_layer& L, uint64_t G, uint64_t k, uint32_t* idx_out, void* ws,
                          cudaStream_t stream) {
  timing_begin(kKernSelect, stream);
  cudaError_t err = cudaSuccess;
  if (k == G) {  // every group is taken: the ascending index list itself
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
  if ((err = cudaMemsetAsync(st, 0, sizeof(SelectState), stream)) != cudaSuccess) return err;
  if ((err = cudaMemsetAsync(hist0, 0, sizeof(uint32_t) * (kSelBins0 + kSelBins1 + kSelBins2), stream)) !=
      cudaSuccess)
    return err;
  norm_hist_kernel<<<lay.ntiles, kSelThreads, 0, stream>>>(L.g, G, L.eta, k, keys, hist0, st);
  hist_refine_kernel<1><<<lay.ntiles, kSelThreads, 0, stream>>>(keys, G, hist1, st);
  hist_refine_kernel<2><<<lay.ntiles, kSelThreads, 0, stream>>>(keys, G, hist2, st);
  tile_count_kernel<<<lay.ntiles, kSelThreads, 0, stream>>>(keys, G, tiles, lay.ntiles, k, st, status);
  scatter_kernel<<<lay.ntiles, kSelThreads, 0, stream>>>(keys, G, tiles, st, k, idx_out);
  err = cudaGetLastError();
  count_launches(5);
  timing_end(kKernSelect, stream);
  return err;
}

}  // namespace pvt
