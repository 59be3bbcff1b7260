// Internal declarations shared by the translation units of libpvt (host side
// launchers, workspace layout, small device helpers).  Not part of the ABI.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "pvt.h"

namespace pvt {

constexpr int kGroupDim = 8;
constexpr int kSmCountFallback = 148;

// ---- workspace layout -------------------------------------------------------
// [0, 256)            header: status word (u32 at 0), selection state, counters
// [256, ...)          region shared by select and encode (they run one after the
//                     other on a stream and never need each other's scratch)
constexpr size_t kWsHeaderBytes = 256;
constexpr size_t kWsAlign = 256;

// selection -------------------------------------------------------------------
constexpr int kSelTile = 4096;      // groups per block of the select kernels
constexpr int kSelThreads = 256;    // 16 groups per thread
constexpr int kSelBins0 = 2048;     // key bits [30:20]
constexpr int kSelBins1 = 2048;     // key bits [19:9]
constexpr int kSelBins2 = 512;      // key bits [8:0]

struct SelectState {        // lives in the header at byte 64
  uint32_t digit0, digit1;  // threshold digits found so far
  uint32_t threshold;       // full threshold key once the last digit is known
  uint32_t need_eq;         // how many groups with key == threshold are taken (lowest indices)
  uint64_t k_left;          // groups still to be taken from the current bucket
  uint32_t done[4];         // block-completion counters of the passes
  uint32_t cand_count;      // keys found inside the threshold bucket of the first digit
};
constexpr size_t kSelStateOffset = 64;

struct SelectLayout {
  size_t hist_off;   // u32 [2048 + 2048 + 512]
  size_t keys_off;   // u32 [G]
  size_t tiles_off;  // u32 [2 * ntiles]: (greater, equal) counts, later exclusive offsets
  size_t cand_off;   // u32 [cand_cap]: keys of the threshold bucket, any order
  uint32_t cand_cap;
  size_t bytes;      // end of the region (from the workspace base)
  uint32_t ntiles;
};
SelectLayout select_layout(uint64_t G);

// encode, M = 1 ---------------------------------------------------------------
// The search kernel leaves, per (target, codebook slice), the sub-chunks of the
// codebook that may hold the nearest codeword; the rescoring kernel evaluates the
// exact distances of those codewords and writes the code.
constexpr int kEncThreads = 256;     // compute threads per CTA (8 warps) + 1 producer warp
constexpr int kChunkCodewords = 256; // codewords per staged chunk (one bulk copy)
constexpr int kSubCodewords = 32;    // tracking granularity of the running minimum
constexpr int kChunkBytes = kChunkCodewords * (kGroupDim * 4 + 4);  // 9216: pairs interleaved + half norms
constexpr int kEncStages = 4;
constexpr int kListLen = 4;          // remembered near-minimum sub-chunks per (target, slice)
constexpr int kMaxSlices = 16;
constexpr uint16_t kCandOverflow = 0xffffu;

struct CandRecord {        // 16 bytes, one per (target, codebook slice)
  float best;              // smallest fast score of the slice
  uint16_t sub[kListLen];  // sub-chunk ids whose minimum lies within the margin of `best`
  uint16_t cnt;            // valid entries of sub[]; kCandOverflow: rescan the whole slice
  uint16_t pad;
};

struct EncodeM1Layout {
  size_t cbx_off;      // expanded codebook: n_chunks * kChunkBytes
  size_t n2max_off;    // u32 bit pattern of max ||c||^2
  size_t gbest_off;    // u32 [k]: order-preserving image of the smallest fast score over all slices
  size_t margin_off;   // f32 [k]: rounding-error margin of the fast score of each target
  size_t rec_off;      // CandRecord [n_tiles][n_slices][tile]
  size_t bytes;
  uint32_t n_chunks;
  uint32_t tile;       // targets per tile (kEncThreads * TT)
  uint32_t n_tiles;
  uint32_t n_slices;   // codebook slices per tile (whole chunks each)
  uint32_t n_ctas;
};
EncodeM1Layout encode_m1_layout(uint32_t K, uint64_t k, int sm_count, int targets_per_thread);
int encode_m1_targets_per_thread(uint64_t k, int sm_count);  // 4 or 8
size_t encode_m2_workspace_bytes();

// encode, M = 1 on the tensor cores (fp16 codebooks of at least 1024 codewords)
struct EncodeM1TcLayout {
  size_t bimg_off;    // codebook image in operand order: n_steps * 4096 bytes
  size_t stats_off;   // max ||c||^2 (bit pattern), exception count
  size_t exc_off;     // u32 [K]: codewords the image cannot represent
  size_t gbest_off, margin_off, rec_off;
  size_t bytes;
  uint32_t n_steps;   // 128-codeword steps
  uint32_t n_tiles;   // tiles of 256 targets
  uint32_t n_slices;
  uint32_t n_ctas;
};
bool encode_m1_use_tc(const pvt_layer& L, uint64_t k);
void set_m1_search(int mode);
EncodeM1TcLayout encode_m1_tc_layout(uint32_t K, uint64_t k, int sm_count, int group_dim = 8);

// launchers (each returns a cudaError_t) --------------------------------------
cudaError_t launch_select(const pvt_layer& L, uint64_t G, uint64_t k, uint32_t* idx_out, void* ws, int sm_count,
                          cudaStream_t stream);
// the same selection on other keys: 0 squared update norm, 1 the same while a straight-through buffer takes the
// step, 2 uniformly random keys, 3 keys of a draw in proportion to the squared update norm (seeded)
cudaError_t launch_select_keyed(const pvt_layer& L, uint64_t G, uint64_t k, uint32_t* idx_out, void* ws, int sm_count,
                                cudaStream_t stream, int key_mode, float* buffer, uint64_t seed);
cudaError_t launch_encode_m1(const pvt_layer& L, uint64_t G, const uint32_t* idx, uint64_t k, float* err_out,
                             void* ws, int sm_count, cudaStream_t stream);
cudaError_t launch_encode_m1_tc(const pvt_layer& L, uint64_t G, const uint32_t* idx, uint64_t k, float* err_out,
                                void* ws, int sm_count, cudaStream_t stream);
cudaError_t launch_encode_m2(const pvt_layer& L, uint64_t G, const uint32_t* idx, uint64_t k, float* err_out,
                             void* ws, int sm_count, cudaStream_t stream);
cudaError_t launch_encode_mx(const pvt_layer& L, uint64_t G, const uint32_t* idx, uint64_t k, float* err_out,
                             void* ws, cudaStream_t stream);
cudaError_t launch_encode_g16(const pvt_layer& L, uint64_t G, const uint32_t* idx, uint64_t k, float* err_out,
                              void* ws, cudaStream_t stream);
cudaError_t launch_dequant(const pvt_layer& L, uint64_t G, void* W_hat, int32_t out_dtype, uint32_t* status,
                           int sm_count, cudaStream_t stream);

cudaError_t launch_pstep_grad(const pvt_layer& L, uint64_t G, double* grad_books, double* grad_scale, uint32_t* status,
                              int sm_count, cudaStream_t stream);
cudaError_t launch_adam(float* param, void* param_f16, const double* grad, float* exp_avg, float* exp_avg_sq,
                        uint64_t n, float lr, float beta1, float beta2, float eps, float bias1, float bias2,
                        int sm_count, cudaStream_t stream);

cudaError_t launch_adam_direction(const float* grad, float* exp_avg, float* exp_avg_sq, float* dir, uint64_t n,
                                  float beta1, float beta2, float eps, float bias1, float bias2, int sm_count,
                                  cudaStream_t stream);

// V step with the subspace size taken from a trust ratio: scratch behind the selection's region
struct TrustLayout {
  size_t idx_off;       // u32 [k]: the selection, ascending
  size_t pairs_a_off;   // u64 [k]: (inverted key, position) pairs; the sorted order ends here
  size_t pairs_b_off;   // u64 [k]: second sort buffer, afterwards f64 [k] squared changes by rank
  size_t counts_off;    // u32 [256 * sort_blocks]
  size_t saved_off;     // u32 [k]: previous codes by position
  size_t partial_off;   // f64 [norm_blocks]
  size_t stats_off;     // f64 [2] + ticket
  size_t encode_off;    // workspace of the search kernels (own header)
  size_t bytes;
  uint32_t sort_blocks, norm_blocks;
};
TrustLayout trust_layout(uint64_t G, uint64_t k, size_t encode_bytes, int sm_count);
cudaError_t launch_trust_rank(const pvt_layer& L, uint64_t G, uint64_t k, void* ws, const TrustLayout& t,
                              cudaStream_t stream);
cudaError_t launch_trust_before_search(const pvt_layer& L, uint64_t G, uint64_t k, void* ws, const TrustLayout& t,
                                       cudaStream_t stream);
cudaError_t launch_trust_after_search(const pvt_layer& L, uint64_t G, uint64_t k, float ratio, uint32_t* idx_out,
                                      uint64_t* n_out, double* stats_out, void* ws, const TrustLayout& t,
                                      cudaStream_t stream);

cudaError_t launch_refine(const pvt_layer& L, uint64_t G, const uint32_t* idx, uint64_t k, int max_moves,
                          float* err_out, uint32_t* moves_out, uint32_t* status, cudaStream_t stream);

// ---- division by an invariant 32-bit divisor ---------------------------------------------------------------
// n / d for every 32-bit n as one multiply-high, a subtraction, an addition and two shifts (Granlund and
// Montgomery, "Division by invariant integers using multiplication", 1994, unsigned case): with l = ceil(log2 d),
// mul = floor(2^32 (2^l - d) / d) + 1, t = mulhi(mul, n):  n / d = (t + ((n - t) >> min(l, 1))) >> max(l - 1, 0).
struct FastDiv {
  uint32_t mul, s1, s2;
};
inline FastDiv make_fast_div(uint32_t d) {
  uint32_t l = 0;
  while (l < 32 && ((uint64_t)1 << l) < d) ++l;
  FastDiv f;
  f.mul = (uint32_t)((((uint64_t)1 << 32) * (((uint64_t)1 << l) - d)) / d + 1);
  f.s1 = l < 1 ? l : 1;
  f.s2 = l > 1 ? l - 1 : 0;
  return f;
}
#ifdef __CUDACC__
__device__ __forceinline__ uint32_t fast_div(uint32_t n, const FastDiv& f) {
  const uint32_t t = __umulhi(f.mul, n);
  return (t + ((n - t) >> f.s1)) >> f.s2;
}
#endif

// ---- programmatic dependent launch --------------------------------------------------------------------
// Consecutive kernels of a call depend on one another, so between two of them the GPU would idle for a launch
// latency.  A kernel launched with launch_dependent() may be scheduled while the kernel before it on the stream
// is still running; it must execute pdl_wait() before its first access to global memory, which returns once
// that kernel has completed and its writes are visible.  Every kernel of a chain calls pdl_trigger() at its
// start to allow the one after it to be scheduled early.  Both are no-ops for a kernel launched the plain way.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t stream,
                             Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

// optional per-kernel timing (benchmark instrumentation) ----------------------
enum KernelId {
  kKernSelect = 0, kKernEncodeMain = 1, kKernEncodeAux = 2, kKernDequant = 3, kKernEncodeRescore = 4,
  kKernPstepGrad = 5, kKernAdam = 6, kKernTrust = 7, kKernRefine = 8, kKernCount = 9
};
void timing_begin(KernelId id, cudaStream_t stream);
void timing_end(KernelId id, cudaStream_t stream);

// remembers the CUDA error behind a PVT_ECUDA return for pvt_last_cuda_error (per host thread)
void record_cuda_error(cudaError_t e);

// multiprocessors of the current device
int device_sm_count();

// number of kernels launched by this process through the library (a claim the benchmark reports)
void count_launches(int n);

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace pvt
