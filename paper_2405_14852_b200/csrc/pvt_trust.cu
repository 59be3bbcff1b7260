// V step whose subspace size follows from a trust ratio (Section 4.3; Appendix J, hyper-parameter paragraph):
// the groups are taken in the order of decreasing update norm and re-encoded, and the longest prefix of that
// order is kept whose total squared change of the dequantised weights stays below ratio^2 * ||W_hat||^2; the
// other groups get their previous codes back; one group always keeps its new code.
//
// The appendix reaches this prefix by re-encoding a hundredth of the weights at a time and undoing the tail of
// the last portion.  Here the k_max groups of largest norm are re-encoded in one go (the search kernels want
// many targets at once), their changes are summed in rank order, and the codes behind the cut are restored:
// the same result whenever the cut falls inside the first k_max groups.
//
// Steps on the stream, after the top-k_max selection (ascending indices):
//   rank_init      key of every selected group (the binary32 norm again, bit for bit) paired with its position
//   4 x radix pass stable LSD sort of the pairs by descending key: positions ascend, so equal norms keep the
//                  lowest index first
//   save_codes     previous codes of the selected groups
//   sq_norm        ||W_hat||^2 of the whole matrix in binary64 (fixed summation tree)
//   search         the library's own encode kernels on the ascending list
//   change         squared change of each group's dequantised weights, stored in rank order
//   cut            running sum in rank order, first position that breaks the bound
//   restore        previous codes for every position from the cut on
#include <cuda_fp16.h>

#include "pvt_internal.h"

namespace pvt {
namespace {

constexpr int kSortThreads = 256;
constexpr int kSortRounds = 8;                          // items per thread
constexpr int kSortTile = kSortThreads * kSortRounds;   // 2048 pairs per block
constexpr int kSortBins = 256;                          // 8 bits per pass, 4 passes over the 32 key bits
constexpr int kSortWarps = kSortThreads / 32;
constexpr int kScanThreads = 1024;
constexpr int kNormThreads = 256;
constexpr int kCutThreads = 1024;

// ---- rank order ------------------------------------------------------------------------------------------------

// pair = (~key) << 32 | position in the ascending index list.  Sorting the pairs by their upper half in ascending
// order, stably, gives (norm descending, index ascending).
template <int DG>
__global__ void __launch_bounds__(256) rank_init_kernel(const float* __restrict__ g, uint64_t G, float eta,
                                                        const uint32_t* __restrict__ idx, uint64_t k,
                                                        uint64_t* __restrict__ pairs, uint32_t* status) {
  const uint64_t a = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (a >= k) return;
  const uint32_t j = __ldg(idx + a);
  uint32_t key = 0;
  if (j < G) {
    const float4* src = reinterpret_cast<const float4*>(g) + (DG / 4) * (size_t)j;
    float acc = 0.0f;
#pragma unroll
    for (int q = 0; q < DG / 4; ++q) {  // one chain over the DG elements in index order
      const float4 x = __ldg(src + q);
      float u;
      u = __fmul_rn(eta, x.x); acc = __fmaf_rn(u, u, acc);
      u = __fmul_rn(eta, x.y); acc = __fmaf_rn(u, u, acc);
      u = __fmul_rn(eta, x.z); acc = __fmaf_rn(u, u, acc);
      u = __fmul_rn(eta, x.w); acc = __fmaf_rn(u, u, acc);
    }
    key = __float_as_uint(acc);
  } else {
    atomicOr(status, PVT_DEV_BAD_INDEX);
  }
  pairs[a] = ((uint64_t)(~key) << 32) | (uint64_t)(uint32_t)a;
}

__device__ __forceinline__ uint32_t digit_of(uint64_t pair, int pass) { return (uint32_t)(pair >> (32 + 8 * pass)) & 255u; }

// counts[bin * n_blocks + block]: how many pairs of this block's tile carry the digit
__global__ void __launch_bounds__(kSortThreads) sort_count_kernel(const uint64_t* __restrict__ in, uint64_t k, int pass,
                                                                  uint32_t* __restrict__ counts, uint32_t n_blocks) {
  __shared__ uint32_t h[kSortBins];
  h[threadIdx.x] = 0;
  __syncthreads();
  const uint64_t base = (uint64_t)blockIdx.x * kSortTile;
#pragma unroll
  for (int r = 0; r < kSortRounds; ++r) {
    const uint64_t p = base + (uint64_t)r * kSortThreads + threadIdx.x;
    if (p < k) atomicAdd(&h[digit_of(in[p], pass)], 1u);
  }
  __syncthreads();
  counts[(size_t)threadIdx.x * n_blocks + blockIdx.x] = h[threadIdx.x];
}

// exclusive prefix sum of n counters in place, one block; every thread owns a contiguous run
__global__ void __launch_bounds__(kScanThreads) sort_scan_kernel(uint32_t* __restrict__ counts, uint32_t n) {
  __shared__ uint32_t part[kScanThreads];
  const uint32_t per = (n + kScanThreads - 1) / kScanThreads;
  const uint32_t lo = threadIdx.x * per, hi = lo + per < n ? lo + per : n;
  uint32_t sum = 0;
  for (uint32_t i = lo; i < hi; ++i) sum += counts[i];
  part[threadIdx.x] = sum;
  __syncthreads();
  for (int off = 1; off < kScanThreads; off <<= 1) {  // inclusive scan of the run totals
    const uint32_t add = threadIdx.x >= (unsigned)off ? part[threadIdx.x - off] : 0u;
    __syncthreads();
    part[threadIdx.x] += add;
    __syncthreads();
  }
  uint32_t run = threadIdx.x ? part[threadIdx.x - 1] : 0u;
  for (uint32_t i = lo; i < hi; ++i) {
    const uint32_t c = counts[i];
    counts[i] = run;
    run += c;
  }
}

// stable scatter: within a block the pairs are visited in position order (round, then thread); a pair's slot is
// the block's start for its digit + the number of earlier pairs of the block with the same digit
__global__ void __launch_bounds__(kSortThreads) sort_scatter_kernel(const uint64_t* __restrict__ in,
                                                                    uint64_t* __restrict__ out, uint64_t k, int pass,
                                                                    const uint32_t* __restrict__ starts,
                                                                    uint32_t n_blocks) {
  __shared__ uint32_t seen[kSortBins];               // pairs of earlier rounds, per digit, plus the block's start
  __shared__ uint32_t cnt[kSortWarps][kSortBins];    // this round: per warp and digit
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  seen[threadIdx.x] = starts[(size_t)threadIdx.x * n_blocks + blockIdx.x];
  const uint64_t base = (uint64_t)blockIdx.x * kSortTile;
  for (int r = 0; r < kSortRounds; ++r) {
#pragma unroll
    for (int w = 0; w < kSortWarps; ++w) cnt[w][threadIdx.x] = 0;
    __syncthreads();
    const uint64_t p = base + (uint64_t)r * kSortThreads + threadIdx.x;
    const bool valid = p < k;
    const uint64_t pair = valid ? in[p] : 0;
    const uint32_t d = valid ? digit_of(pair, pass) : kSortBins;  // past the end: a digit of its own
    const uint32_t peers = __match_any_sync(0xffffffffu, d);
    const uint32_t before = __popc(peers & ((1u << lane) - 1u));
    if (valid && before == 0) cnt[warp][d] = __popc(peers);
    __syncthreads();
    {  // thread = digit: turn the per-warp counts into offsets, advance the running total
      uint32_t run = seen[threadIdx.x];
#pragma unroll
      for (int w = 0; w < kSortWarps; ++w) {
        const uint32_t c = cnt[w][threadIdx.x];
        cnt[w][threadIdx.x] = run;
        run += c;
      }
      seen[threadIdx.x] = run;
    }
    __syncthreads();
    if (valid) {
      const uint32_t slot = cnt[warp][d] + before;
      if (slot < k) out[slot] = pair;
    }
    __syncthreads();
  }
}

// ---- codes and dequantised values ------------------------------------------------------------------------------

// codes of a group packed into one word: the two-byte code itself for two-byte codes (one codebook), otherwise
// byte m = code of codebook m
template <bool CODE_U16>
__device__ __forceinline__ uint32_t load_codes(const void* codes, uint32_t j, int M) {
  if (CODE_U16) return reinterpret_cast<const uint16_t*>(codes)[j];  // M == 1
  if (M == 2) return reinterpret_cast<const uint16_t*>(codes)[j];    // two adjacent bytes: first | second << 8
  const uint8_t* c = reinterpret_cast<const uint8_t*>(codes) + (size_t)j * M;
  uint32_t packed = 0;
  for (int m = 0; m < M; ++m) packed |= (uint32_t)c[m] << (8 * m);
  return packed;
}

template <bool CODE_U16>
__device__ __forceinline__ void store_codes(void* codes, uint32_t j, int M, uint32_t packed) {
  if (CODE_U16 || M == 2) {
    reinterpret_cast<uint16_t*>(codes)[j] = (uint16_t)packed;
  } else {
    uint8_t* c = reinterpret_cast<uint8_t*>(codes) + (size_t)j * M;
    for (int m = 0; m < M; ++m) c[m] = (uint8_t)(packed >> (8 * m));
  }
}

template <bool CB_F16, int DG>
__device__ __forceinline__ void codeword(const void* book, uint32_t code, float* c) {
  if (CB_F16) {
#pragma unroll
    for (int part = 0; part < DG / 8; ++part) {
      const uint4 raw = __ldg(reinterpret_cast<const uint4*>(book) + (size_t)code * (DG / 8) + part);
      const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
        c[8 * part + 2 * i] = f.x;
        c[8 * part + 2 * i + 1] = f.y;
      }
    }
  } else {
    const float4* src = reinterpret_cast<const float4*>(book) + (size_t)code * (DG / 4);
#pragma unroll
    for (int part = 0; part < DG / 4; ++part) {
      const float4 x = __ldg(src + part);
      c[4 * part] = x.x, c[4 * part + 1] = x.y, c[4 * part + 2] = x.z, c[4 * part + 3] = x.w;
    }
  }
}

// the dequantised weights of a group, binary32 exactly as dequantisation forms them: v = c1 (+ c2 ...), w = s * v
template <bool CB_F16, int DG>
__device__ __forceinline__ bool group_weights(const void* books, uint32_t K, int M, uint32_t packed, bool code_u16,
                                              float s, float* w) {
  const uint32_t b0 = (M >= 2 && !code_u16) ? (packed & 0xffu) : packed;
  bool ok = b0 < K;
  for (int m = 1; m < M; ++m) ok = ok && ((packed >> (8 * m)) & 0xffu) < K;
  float v[DG];
  codeword<CB_F16, DG>(books, ok ? b0 : 0, v);
  for (int m = 1; m < M; ++m) {  // codebooks added left to right, each sum rounded once
    float v2[DG];
    codeword<CB_F16, DG>(books, (uint32_t)m * K + (ok ? ((packed >> (8 * m)) & 0xffu) : 0u), v2);
#pragma unroll
    for (int i = 0; i < DG; ++i) v[i] = __fadd_rn(v[i], v2[i]);
  }
#pragma unroll
  for (int i = 0; i < DG; ++i) w[i] = __fmul_rn(s, v[i]);
  return ok;
}

struct TrustParams {
  const void* books;
  void* codes;
  const float* scale;
  uint64_t G, k;
  uint32_t gpr, K;
  int M;
  const uint32_t* idx;      // ascending list of the selection [k]
  const uint64_t* pairs;    // sorted pairs [k]: lower half = position in idx
  uint32_t* saved;          // previous codes by position [k]
  double* change;           // squared change by rank [k]
  uint32_t* rank_idx;       // group index by rank [k] (caller's output)
  double* partial;          // per-block sums of the norm kernel
  uint32_t* ticket;
  double* stats;            // [0] ||W_hat||^2, [1] total squared change of the kept groups
  uint64_t* n_out;
  float ratio;
  uint32_t* status;
  const uint32_t* enc_status;
};

template <bool CODE_U16>
__global__ void __launch_bounds__(256) save_codes_kernel(const TrustParams p) {
  const uint64_t a = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (a >= p.k) return;
  const uint32_t j = __ldg(p.idx + a);
  p.saved[a] = j < p.G ? load_codes<CODE_U16>(p.codes, j, p.M) : 0u;
}

// ||W_hat||^2: every thread adds its groups in index order, the block adds its threads in a fixed tree, the last
// block to finish adds the block sums in block order -- the same binary64 result on every run
template <bool CB_F16, bool CODE_U16, int DG>
__global__ void __launch_bounds__(kNormThreads) sq_norm_kernel(const TrustParams p) {
  __shared__ double sh[kNormThreads];
  __shared__ bool last;
  double acc = 0.0;
  bool bad = false;
  const uint64_t stride = (uint64_t)gridDim.x * kNormThreads;
  for (uint64_t j = (uint64_t)blockIdx.x * kNormThreads + threadIdx.x; j < p.G; j += stride) {
    float w[DG];
    const uint32_t packed = load_codes<CODE_U16>(p.codes, (uint32_t)j, p.M);
    bad |= !group_weights<CB_F16, DG>(p.books, p.K, p.M, packed, CODE_U16, __ldg(p.scale + (uint32_t)j / p.gpr), w);
#pragma unroll
    for (int i = 0; i < DG; ++i) acc = __fma_rn((double)w[i], (double)w[i], acc);
  }
  if (bad) atomicOr(p.status, PVT_DEV_BAD_CODE);
  sh[threadIdx.x] = acc;
  __syncthreads();
  for (int off = kNormThreads / 2; off > 0; off >>= 1) {
    if (threadIdx.x < off) sh[threadIdx.x] += sh[threadIdx.x + off];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    p.partial[blockIdx.x] = sh[0];
    __threadfence();
    last = atomicAdd(p.ticket, 1u) == gridDim.x - 1;
  }
  __syncthreads();
  if (last && threadIdx.x == 0) {
    __threadfence();
    double total = 0.0;
    for (unsigned b = 0; b < gridDim.x; ++b) total += *(volatile double*)&p.partial[b];
    p.stats[0] = total;
    *p.ticket = 0;
  }
}

// squared change of the dequantised weights of the group at every rank; the group index in rank order
template <bool CB_F16, bool CODE_U16, int DG>
__global__ void __launch_bounds__(256) change_kernel(const TrustParams p) {
  const uint64_t r = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= p.k) return;
  const uint32_t a = (uint32_t)p.pairs[r];
  uint32_t j = a < p.k ? __ldg(p.idx + a) : 0xffffffffu;
  double acc = 0.0;
  if (j < p.G) {
    const float s = __ldg(p.scale + j / p.gpr);
    float wo[DG], wn[DG];
    bool ok = group_weights<CB_F16, DG>(p.books, p.K, p.M, p.saved[a], CODE_U16, s, wo);
    ok &= group_weights<CB_F16, DG>(p.books, p.K, p.M, load_codes<CODE_U16>(p.codes, j, p.M), CODE_U16, s, wn);
    if (!ok) atomicOr(p.status, PVT_DEV_BAD_CODE);
#pragma unroll
    for (int i = 0; i < DG; ++i) {
      const double diff = __dsub_rn((double)wn[i], (double)wo[i]);
      acc = __dadd_rn(acc, __dmul_rn(diff, diff));
    }
  } else {
    j = 0;
  }
  p.change[r] = acc;
  p.rank_idx[r] = j;
}

// One block.  Running sum of the changes in rank order (each thread owns a contiguous run; the run totals are
// added in order by one thread); n = first rank whose running sum is not below ratio^2 * ||W_hat||^2, at least 1.
__global__ void __launch_bounds__(kCutThreads) cut_kernel(const TrustParams p) {
  __shared__ double run_start[kCutThreads];
  __shared__ unsigned long long first_bad;
  const uint64_t per = (p.k + kCutThreads - 1) / kCutThreads;
  const uint64_t lo = threadIdx.x * per, hi = lo + per < p.k ? lo + per : p.k;
  double sum = 0.0;
  for (uint64_t r = lo; r < hi; ++r) sum += p.change[r];
  run_start[threadIdx.x] = sum;
  if (threadIdx.x == 0) first_bad = p.k;
  __syncthreads();
  if (threadIdx.x == 0) {
    double run = 0.0;
    for (int t = 0; t < kCutThreads; ++t) {
      const double s = run_start[t];
      run_start[t] = run;
      run += s;
    }
  }
  __syncthreads();
  const double limit = ((double)p.ratio * (double)p.ratio) * p.stats[0];
  double run = run_start[threadIdx.x];
  for (uint64_t r = lo; r < hi; ++r) {
    run += p.change[r];
    if (!(run < limit)) {
      atomicMin(&first_bad, (unsigned long long)r);
      break;
    }
  }
  __syncthreads();
  const uint64_t n = first_bad < 1 ? 1 : first_bad;  // one change always goes through
  if (lo < n && n <= hi) {  // the thread that owns rank n - 1 reports the change that was let through
    double kept = run_start[threadIdx.x];
    for (uint64_t r = lo; r < n; ++r) kept += p.change[r];
    p.stats[1] = kept;
  }
  if (threadIdx.x == 0) {
    *p.n_out = n;
    const uint32_t e = *p.enc_status;
    if (e) atomicOr(p.status, e);
  }
}

template <bool CODE_U16>
__global__ void __launch_bounds__(256) restore_kernel(const TrustParams p) {
  const uint64_t r = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= p.k || r < *p.n_out) return;
  const uint32_t a = (uint32_t)p.pairs[r];
  const uint32_t j = p.rank_idx[r];
  if (a < p.k && j < p.G) store_codes<CODE_U16>(p.codes, j, p.M, p.saved[a]);
}

size_t host_align(size_t x) { return (x + kWsAlign - 1) & ~(kWsAlign - 1); }

}  // namespace

TrustLayout trust_layout(uint64_t G, uint64_t k, size_t encode_bytes, int sm_count) {
  TrustLayout t;
  t.sort_blocks = (uint32_t)((k + kSortTile - 1) / kSortTile);
  t.norm_blocks = (uint32_t)(4 * (sm_count > 0 ? sm_count : kSmCountFallback));
  t.idx_off = host_align(select_layout(G).bytes);
  t.pairs_a_off = host_align(t.idx_off + sizeof(uint32_t) * k);
  t.pairs_b_off = host_align(t.pairs_a_off + sizeof(uint64_t) * k);   // second sort buffer, later the changes
  t.counts_off = host_align(t.pairs_b_off + sizeof(uint64_t) * k);
  t.saved_off = host_align(t.counts_off + sizeof(uint32_t) * kSortBins * (size_t)t.sort_blocks);
  t.partial_off = host_align(t.saved_off + sizeof(uint32_t) * k);
  t.stats_off = host_align(t.partial_off + sizeof(double) * t.norm_blocks);  // stats[2], ticket
  t.encode_off = host_align(t.stats_off + 64);
  t.bytes = t.encode_off + host_align(encode_bytes);
  return t;
}

cudaError_t launch_trust_rank(const pvt_layer& L, uint64_t G, uint64_t k, void* ws, const TrustLayout& t,
                              cudaStream_t stream) {
  char* base = static_cast<char*>(ws);
  uint32_t* status = reinterpret_cast<uint32_t*>(base);
  const uint32_t* idx = reinterpret_cast<const uint32_t*>(base + t.idx_off);
  uint64_t* a = reinterpret_cast<uint64_t*>(base + t.pairs_a_off);
  uint64_t* b = reinterpret_cast<uint64_t*>(base + t.pairs_b_off);
  uint32_t* counts = reinterpret_cast<uint32_t*>(base + t.counts_off);
  const unsigned flat = (unsigned)((k + 255) / 256);
  if (L.group_dim == 16)
    rank_init_kernel<16><<<flat, 256, 0, stream>>>(L.g, G, L.eta, idx, k, a, status);
  else
    rank_init_kernel<8><<<flat, 256, 0, stream>>>(L.g, G, L.eta, idx, k, a, status);
  for (int pass = 0; pass < 4; ++pass) {
    sort_count_kernel<<<t.sort_blocks, kSortThreads, 0, stream>>>(a, k, pass, counts, t.sort_blocks);
    sort_scan_kernel<<<1, kScanThreads, 0, stream>>>(counts, kSortBins * t.sort_blocks);
    sort_scatter_kernel<<<t.sort_blocks, kSortThreads, 0, stream>>>(a, b, k, pass, counts, t.sort_blocks);
    uint64_t* tmp = a;
    a = b;
    b = tmp;
  }
  count_launches(13);
  return cudaGetLastError();
}

namespace {

TrustParams make_params(const pvt_layer& L, uint64_t G, uint64_t k, float ratio, uint32_t* idx_out, uint64_t* n_out,
                        void* ws, const TrustLayout& t) {
  char* base = static_cast<char*>(ws);
  TrustParams p;
  p.books = L.codebooks;
  p.codes = L.codes;
  p.scale = L.scale;
  p.G = G;
  p.k = k;
  p.gpr = (uint32_t)(L.cols / L.group_dim);
  p.K = (uint32_t)L.codebook_size;
  p.M = L.num_codebooks;
  p.idx = reinterpret_cast<const uint32_t*>(base + t.idx_off);
  p.pairs = reinterpret_cast<const uint64_t*>(base + t.pairs_a_off);  // four passes end in the first buffer
  p.saved = reinterpret_cast<uint32_t*>(base + t.saved_off);
  p.change = reinterpret_cast<double*>(base + t.pairs_b_off);
  p.rank_idx = idx_out;
  p.partial = reinterpret_cast<double*>(base + t.partial_off);
  p.stats = reinterpret_cast<double*>(base + t.stats_off);
  p.ticket = reinterpret_cast<uint32_t*>(base + t.stats_off + 2 * sizeof(double));
  p.n_out = n_out;
  p.ratio = ratio;
  p.status = reinterpret_cast<uint32_t*>(base);
  p.enc_status = reinterpret_cast<const uint32_t*>(base + t.encode_off);
  return p;
}

template <bool CB_F16, bool CODE_U16>
cudaError_t before_search(const TrustParams& p, int dg, unsigned norm_blocks, cudaStream_t stream) {
  const unsigned flat = (unsigned)((p.k + 255) / 256);
  save_codes_kernel<CODE_U16><<<flat, 256, 0, stream>>>(p);
  if (dg == 16)
    sq_norm_kernel<CB_F16, CODE_U16, 16><<<norm_blocks, kNormThreads, 0, stream>>>(p);
  else
    sq_norm_kernel<CB_F16, CODE_U16, 8><<<norm_blocks, kNormThreads, 0, stream>>>(p);
  count_launches(2);
  return cudaGetLastError();
}

template <bool CB_F16, bool CODE_U16>
cudaError_t after_search(const TrustParams& p, int dg, cudaStream_t stream) {
  const unsigned flat = (unsigned)((p.k + 255) / 256);
  if (dg == 16)
    change_kernel<CB_F16, CODE_U16, 16><<<flat, 256, 0, stream>>>(p);
  else
    change_kernel<CB_F16, CODE_U16, 8><<<flat, 256, 0, stream>>>(p);
  cut_kernel<<<1, kCutThreads, 0, stream>>>(p);
  restore_kernel<CODE_U16><<<flat, 256, 0, stream>>>(p);
  count_launches(3);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_trust_before_search(const pvt_layer& L, uint64_t G, uint64_t k, void* ws, const TrustLayout& t,
                                       cudaStream_t stream) {
  const TrustParams p = make_params(L, G, k, 0.0f, nullptr, nullptr, ws, t);
  cudaError_t e = cudaMemsetAsync(static_cast<char*>(ws) + t.stats_off, 0, 64, stream);
  if (e != cudaSuccess) return e;
  const bool f16 = L.codebook_dtype == PVT_F16, u16 = L.code_dtype == PVT_U16;
  const int dg = L.group_dim;
  if (f16)
    return u16 ? before_search<true, true>(p, dg, t.norm_blocks, stream)
               : before_search<true, false>(p, dg, t.norm_blocks, stream);
  return u16 ? before_search<false, true>(p, dg, t.norm_blocks, stream)
             : before_search<false, false>(p, dg, t.norm_blocks, stream);
}

cudaError_t launch_trust_after_search(const pvt_layer& L, uint64_t G, uint64_t k, float ratio, uint32_t* idx_out,
                                      uint64_t* n_out, double* stats_out, void* ws, const TrustLayout& t,
                                      cudaStream_t stream) {
  const TrustParams p = make_params(L, G, k, ratio, idx_out, n_out, ws, t);
  const bool f16 = L.codebook_dtype == PVT_F16, u16 = L.code_dtype == PVT_U16;
  cudaError_t e;
  if (f16)
    e = u16 ? after_search<true, true>(p, L.group_dim, stream) : after_search<true, false>(p, L.group_dim, stream);
  else
    e = u16 ? after_search<false, true>(p, L.group_dim, stream) : after_search<false, false>(p, L.group_dim, stream);
  if (e == cudaSuccess && stats_out)
    e = cudaMemcpyAsync(stats_out, p.stats, 2 * sizeof(double), cudaMemcpyDeviceToDevice, stream);
  return e;
}

}  // namespace pvt
