// Host side of the C ABI: argument validation, workspace sizing, status word,
// optional per-kernel timing.  Everything here runs on the host and only enqueues
// work; the arithmetic of the V step lives in the kernels of the other files.
#include <atomic>
#include <cmath>
#include <mutex>
#include <vector>

#include "pvt_encode_m1.cuh"
#include "pvt_internal.h"

namespace pvt {
namespace {

thread_local cudaError_t g_last_cuda = cudaSuccess;
std::atomic<unsigned long long> g_launches{0};

int fail_cuda(cudaError_t e) {
  g_last_cuda = e;
  return PVT_ECUDA;
}

int sm_count() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
      n <= 0) {
    (void)cudaGetLastError();
    return kSmCountFallback;
  }
  return n;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }  // true for NULL

// codes are read two bytes at a time when they are two-byte codes, or a pair of one-byte codes
bool codes_aligned(const pvt_layer* L) {
  const bool two_byte_access = L->code_dtype == PVT_U16 || L->num_codebooks == 2;
  return !two_byte_access || (reinterpret_cast<uintptr_t>(L->codes) & 1u) == 0;
}

// Shape / type checks shared by every entry point.  Returns PVT_OK and G, or the error.
int check_layer(const pvt_layer* L, uint64_t* G_out) {
  if (!L) return PVT_EINVAL;
  if (L->rows <= 0 || L->cols <= 0) return PVT_EINVAL;
  if (L->group_dim != 8 && L->group_dim != 16) return L->group_dim > 0 ? PVT_EUNSUPPORTED : PVT_EINVAL;
  if (L->cols % L->group_dim != 0) return PVT_EINVAL;
  const uint64_t G = (uint64_t)L->rows * (uint64_t)(L->cols / L->group_dim);
  if (G >= (1ull << 32)) return PVT_EINVAL;
  if (!(L->eta >= 0.0f) || !(L->eta <= 3.0e38f)) return PVT_EINVAL;
  *G_out = G;
  return PVT_OK;
}

int check_quantiser(const pvt_layer* L) {
  const int M = L->num_codebooks, K = L->codebook_size;
  if (M < 1 || K < 1) return PVT_EINVAL;
  if (L->codebook_dtype != PVT_F32 && L->codebook_dtype != PVT_F16) return PVT_EINVAL;
  if (L->code_dtype != PVT_U8 && L->code_dtype != PVT_U16) return PVT_EINVAL;
  if (M > 4 || K < 2) return PVT_EUNSUPPORTED;
  if (M == 1 && K > 65536) return PVT_EUNSUPPORTED;
  if (L->code_dtype == PVT_U8 && K > 256) return PVT_EINVAL;
  if (M >= 2 && K > 256) return PVT_EUNSUPPORTED;
  if (M >= 3 && L->code_dtype != PVT_U8) return PVT_EUNSUPPORTED;
  if (L->group_dim == 16 && M != 1) return PVT_EUNSUPPORTED;  // groups of 16 weights: one codebook
  return PVT_OK;
}

// ---- optional timing ----------------------------------------------------------
struct Timing {
  std::mutex mu;
  bool enabled = false;
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> spans[kKernCount];
  cudaEvent_t open[kKernCount] = {};
};
Timing& timing() {
  static Timing t;
  return t;
}

}  // namespace

void record_cuda_error(cudaError_t e) { g_last_cuda = e; }

int device_sm_count() { return sm_count(); }

void count_launches(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

void timing_begin(KernelId id, cudaStream_t stream) {
  Timing& t = timing();
  if (!t.enabled) return;
  std::lock_guard<std::mutex> lock(t.mu);
  cudaEvent_t a;
  if (cudaEventCreate(&a) != cudaSuccess) return;
  cudaEventRecord(a, stream);
  t.open[id] = a;
}

void timing_end(KernelId id, cudaStream_t stream) {
  Timing& t = timing();
  if (!t.enabled) return;
  std::lock_guard<std::mutex> lock(t.mu);
  if (!t.open[id]) return;
  cudaEvent_t b;
  if (cudaEventCreate(&b) != cudaSuccess) return;
  cudaEventRecord(b, stream);
  t.spans[id].push_back({t.open[id], b});
  t.open[id] = nullptr;
}

}  // namespace pvt

namespace pvt {
// 16 independent chains of dependent FMAs per thread: nothing but the FP32 pipe is busy
__global__ void __launch_bounds__(256) ffma_probe_kernel(float* out, int iters) {
  float x[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) x[i] = 1.0f + 1e-3f * (float)(threadIdx.x + i);
  const float a = 1.0000001f, b = 1e-7f;
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < 16; ++i) x[i] = __fmaf_rn(x[i], a, b);
  }
  float s = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; ++i) s += x[i];
  out[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = s;
}

}  // namespace pvt

using namespace pvt;

namespace {

// workspace of pvt_vstep_encode for k groups of this layer
size_t encode_bytes(const pvt_layer& L, uint64_t k, int sms) {
  if (L.num_codebooks >= 3) return encode_m2_workspace_bytes();  // header + the codebooks' image
  if (L.group_dim == 16)
    return encode_m1_use_tc(L, k) ? encode_m1_tc_layout((uint32_t)L.codebook_size, k, sms, 16).bytes : kWsHeaderBytes;
  if (L.num_codebooks != 1) return encode_m2_workspace_bytes();
  return encode_m1_use_tc(L, k)
             ? encode_m1_tc_layout((uint32_t)L.codebook_size, k, sms).bytes
             : encode_m1_layout((uint32_t)L.codebook_size, k, sms, encode_m1_targets_per_thread(k, sms)).bytes;
}

}  // namespace

extern "C" {

size_t pvt_workspace_bytes(const pvt_layer* layer, uint64_t k) {
  uint64_t G = 0;
  if (check_layer(layer, &G) != PVT_OK || check_quantiser(layer) != PVT_OK) return 0;
  if (k < 1 || k > G) return 0;
  const size_t s = select_layout(G).bytes, e = encode_bytes(*layer, k, sm_count());
  return e > s ? e : s;
}

size_t pvt_trust_workspace_bytes(const pvt_layer* layer, uint64_t k_max) {
  uint64_t G = 0;
  if (check_layer(layer, &G) != PVT_OK || check_quantiser(layer) != PVT_OK) return 0;
  if (k_max < 1 || k_max > G) return 0;
  const int sms = sm_count();
  return trust_layout(G, k_max, encode_bytes(*layer, k_max, sms), sms).bytes;
}

int pvt_workspace_init(void* ws, size_t ws_bytes, void* cuda_stream) {
  if (!ws || ws_bytes < kWsHeaderBytes || (reinterpret_cast<uintptr_t>(ws) & (kWsAlign - 1))) return PVT_EINVAL;
  const cudaError_t e = cudaMemsetAsync(ws, 0, kWsHeaderBytes, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? PVT_OK : fail_cuda(e);
}

int pvt_vstep_select(const pvt_layer* layer, uint64_t k, uint32_t* idx_out, void* ws, size_t ws_bytes,
                     void* cuda_stream) {
  uint64_t G = 0;
  int rc = check_layer(layer, &G);
  if (rc != PVT_OK) return rc;
  if (k < 1 || k > G) return PVT_EINVAL;
  if (!layer->g || !aligned16(layer->g) || !idx_out || !aligned4(idx_out) || !ws) return PVT_EINVAL;
  if (reinterpret_cast<uintptr_t>(ws) & (kWsAlign - 1)) return PVT_EINVAL;
  if (ws_bytes < select_layout(G).bytes) return PVT_EWORKSPACE;
  const cudaError_t e = launch_select(*layer, G, k, idx_out, ws, sm_count(), static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? PVT_OK : fail_cuda(e);
}

int pvt_vstep_select_ste(const pvt_layer* layer, float* buffer, uint64_t k, uint32_t* idx_out, void* ws,
                         size_t ws_bytes, void* cuda_stream) {
  uint64_t G = 0;
  int rc = check_layer(layer, &G);
  if (rc != PVT_OK) return rc;
  if (k < 1 || k > G) return PVT_EINVAL;
  if (!layer->g || !aligned16(layer->g) || !buffer || !aligned16(buffer) || !idx_out || !aligned4(idx_out) || !ws)
    return PVT_EINVAL;
  if (static_cast<const void*>(buffer) == static_cast<const void*>(layer->g)) return PVT_EINVAL;
  if (reinterpret_cast<uintptr_t>(ws) & (kWsAlign - 1)) return PVT_EINVAL;
  if (ws_bytes < select_layout(G).bytes) return PVT_EWORKSPACE;
  const cudaError_t e = launch_select_keyed(*layer, G, k, idx_out, ws, sm_count(),
                                            static_cast<cudaStream_t>(cuda_stream), 1, buffer, 0);
  return e == cudaSuccess ? PVT_OK : fail_cuda(e);
}

int pvt_vstep_sample(const pvt_layer* layer, uint64_t k, int32_t rule, uint64_t seed, uint32_t* idx_out, void* ws,
                     size_t ws_bytes, void* cuda_stream) {
  uint64_t G = 0;
  int rc = check_layer(layer, &G);
  if (rc != PVT_OK) return rc;
  if (rule != PVT_SAMPLE_UNIFORM && rule != PVT_SAMPLE_PROPORTIONAL) return PVT_EINVAL;
  if (k < 1 || k > G) return PVT_EINVAL;
  if (rule == PVT_SAMPLE_PROPORTIONAL && (!layer->g || !aligned16(layer->g))) return PVT_EINVAL;
  if (!idx_out || !aligned4(idx_out) || !ws) return PVT_EINVAL;
  if (reinterpret_cast<uintptr_t>(ws) & (kWsAlign - 1)) return PVT_EINVAL;
  if (ws_bytes < select_layout(G).bytes) return PVT_EWORKSPACE;
  const cudaError_t e = launch_select_keyed(*layer, G, k, idx_out, ws, sm_count(),
                                            static_cast<cudaStream_t>(cuda_stream),
                                            rule == PVT_SAMPLE_UNIFORM ? 2 : 3, nullptr, seed);
  return e == cudaSuccess ? PVT_OK : fail_cuda(e);
}

int pvt_vstep_encode(const pvt_layer* layer, const uint32_t* idx, uint64_t k, float* err_out, void* ws,
                     size_t ws_bytes, void* cuda_stream) {
  uint64_t G = 0;
  int rc = check_layer(layer, &G);
  if (rc != PVT_OK) return rc;
  if ((rc = check_quantiser(layer)) != PVT_OK) return rc;
  if (k < 1 || k > G) return PVT_EINVAL;
  if (!layer->W || !layer->g || !layer->scale || !layer->codebooks || !layer->codes || !idx || !ws) return PVT_EINVAL;
  if (!aligned16(layer->W) || !aligned16(layer->g) || !aligned16(layer->codebooks)) return PVT_EINVAL;
  if (!codes_aligned(layer) || !aligned4(idx) || !aligned4(err_out)) return PVT_EINVAL;
  if (reinterpret_cast<uintptr_t>(ws) & (kWsAlign - 1)) return PVT_EINVAL;
  const int sms = sm_count();
  cudaError_t e;
  if (layer->group_dim == 16 && !encode_m1_use_tc(*layer, k)) {
    if (ws_bytes < kWsHeaderBytes) return PVT_EWORKSPACE;
    e = launch_encode_g16(*layer, G, idx, k, err_out, ws, static_cast<cudaStream_t>(cuda_stream));
  } else if (layer->group_dim == 16) {
    if (ws_bytes < encode_m1_tc_layout((uint32_t)layer->codebook_size, k, sms, 16).bytes) return PVT_EWORKSPACE;
    e = launch_encode_m1_tc(*layer, G, idx, k, err_out, ws, sms, static_cast<cudaStream_t>(cuda_stream));
  } else if (layer->num_codebooks == 1 && encode_m1_use_tc(*layer, k)) {
    if (ws_bytes < encode_m1_tc_layout((uint32_t)layer->codebook_size, k, sms).bytes) return PVT_EWORKSPACE;
    e = launch_encode_m1_tc(*layer, G, idx, k, err_out, ws, sms, static_cast<cudaStream_t>(cuda_stream));
  } else if (layer->num_codebooks == 1) {
    const EncodeM1Layout lay =
        encode_m1_layout((uint32_t)layer->codebook_size, k, sms, encode_m1_targets_per_thread(k, sms));
    if (ws_bytes < lay.bytes) return PVT_EWORKSPACE;
    e = launch_encode_m1(*layer, G, idx, k, err_out, ws, sms, static_cast<cudaStream_t>(cuda_stream));
  } else if (layer->num_codebooks == 2) {
    if (layer->code_dtype != PVT_U8) return PVT_EUNSUPPORTED;
    if (layer->beam < 1 || layer->beam > 8) return PVT_EUNSUPPORTED;
    if (ws_bytes < encode_m2_workspace_bytes()) return PVT_EWORKSPACE;
    e = launch_encode_m2(*layer, G, idx, k, err_out, ws, sms, static_cast<cudaStream_t>(cuda_stream));
  } else {
    if (layer->beam < 1 || layer->beam > 8) return PVT_EUNSUPPORTED;
    if (ws_bytes < encode_m2_workspace_bytes()) return PVT_EWORKSPACE;
    e = launch_encode_mx(*layer, G, idx, k, err_out, ws, static_cast<cudaStream_t>(cuda_stream));
  }
  return e == cudaSuccess ? PVT_OK : fail_cuda(e);
}

int pvt_vstep_trust(const pvt_layer* layer, uint64_t k_max, float ratio, uint32_t* idx_out, uint64_t* n_out,
                    double* stats_out, void* ws, size_t ws_bytes, void* cuda_stream) {
  uint64_t G = 0;
  int rc = check_layer(layer, &G);
  if (rc != PVT_OK) return rc;
  if ((rc = check_quantiser(layer)) != PVT_OK) return rc;
  if (k_max < 1 || k_max > G) return PVT_EINVAL;
  if (!(ratio >= 0.0f) || !(ratio <= 3.0e38f)) return PVT_EINVAL;
  if (!layer->W || !layer->g || !layer->scale || !layer->codebooks || !layer->codes || !idx_out || !n_out || !ws)
    return PVT_EINVAL;
  if (!aligned16(layer->W) || !aligned16(layer->g) || !aligned16(layer->codebooks)) return PVT_EINVAL;
  if ((reinterpret_cast<uintptr_t>(n_out) & 7u) || (reinterpret_cast<uintptr_t>(stats_out) & 7u)) return PVT_EINVAL;
  if (!codes_aligned(layer) || !aligned4(idx_out)) return PVT_EINVAL;
  if (reinterpret_cast<uintptr_t>(ws) & (kWsAlign - 1)) return PVT_EINVAL;
  if (layer->num_codebooks >= 2) {
    if (layer->code_dtype != PVT_U8 || layer->beam < 1 || layer->beam > 8) return PVT_EUNSUPPORTED;
    if (layer->num_codebooks == 2 && (reinterpret_cast<uintptr_t>(layer->codes) & 1u)) return PVT_EINVAL;
  }
  const int sms = sm_count();
  const TrustLayout t = trust_layout(G, k_max, encode_bytes(*layer, k_max, sms), sms);
  if (ws_bytes < t.bytes) return PVT_EWORKSPACE;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  char* base = static_cast<char*>(ws);
  uint32_t* idx_sel = reinterpret_cast<uint32_t*>(base + t.idx_off);
  cudaError_t e = launch_select(*layer, G, k_max, idx_sel, ws, sms, stream);
  timing_begin(kKernTrust, stream);
  if (e == cudaSuccess) e = launch_trust_rank(*layer, G, k_max, ws, t, stream);
  if (e == cudaSuccess) e = launch_trust_before_search(*layer, G, k_max, ws, t, stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(base + t.encode_off, 0, kWsHeaderBytes, stream);
  timing_end(kKernTrust, stream);
  if (e != cudaSuccess) return fail_cuda(e);
  rc = pvt_vstep_encode(layer, idx_sel, k_max, nullptr, base + t.encode_off, t.bytes - t.encode_off, cuda_stream);
  if (rc != PVT_OK) return rc;
  e = launch_trust_after_search(*layer, G, k_max, ratio, idx_out, n_out, stats_out, ws, t, stream);
  return e == cudaSuccess ? PVT_OK : fail_cuda(e);
}

int pvt_vstep_refine(const pvt_layer* layer, const uint32_t* idx, uint64_t k, int32_t max_moves, float* err_out,
                     uint32_t* moves_out, uint32_t* status, void* cuda_stream) {
  uint64_t G = 0;
  int rc = check_layer(layer, &G);
  if (rc != PVT_OK) return rc;
  if ((rc = check_quantiser(layer)) != PVT_OK) return rc;
  if (k < 1 || k > G || max_moves < 0 || max_moves > 65535) return PVT_EINVAL;
  if (!layer->W || !layer->g || !layer->scale || !layer->codebooks || !layer->codes || !idx) return PVT_EINVAL;
  if (!aligned16(layer->W) || !aligned16(layer->g) || !aligned16(layer->codebooks)) return PVT_EINVAL;
  if (layer->group_dim != kGroupDim) return PVT_EUNSUPPORTED;
  if (layer->num_codebooks >= 2 && layer->code_dtype != PVT_U8) return PVT_EUNSUPPORTED;
  if (!codes_aligned(layer) || !aligned4(idx) || !aligned4(err_out) || !aligned4(moves_out) || !aligned4(status))
    return PVT_EINVAL;
  const cudaError_t e = launch_refine(*layer, G, idx, k, max_moves, err_out, moves_out, status,
                                      static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? PVT_OK : fail_cuda(e);
}

int pvt_dequant(const pvt_layer* layer, void* W_hat, int32_t out_dtype, uint32_t* status, void* cuda_stream) {
  uint64_t G = 0;
  int rc = check_layer(layer, &G);
  if (rc != PVT_OK) return rc;
  if ((rc = check_quantiser(layer)) != PVT_OK) return rc;
  if (out_dtype != PVT_F32 && out_dtype != PVT_F16) return PVT_EINVAL;
  if (!layer->scale || !layer->codebooks || !layer->codes || !W_hat) return PVT_EINVAL;
  if (!aligned16(layer->codebooks) || !aligned16(W_hat)) return PVT_EINVAL;
  if (!codes_aligned(layer) || !aligned4(status)) return PVT_EINVAL;
  const cudaError_t e = launch_dequant(*layer, G, W_hat, out_dtype, status, sm_count(), static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? PVT_OK : fail_cuda(e);
}

size_t pvt_block_workspace_bytes(const pvt_layer* layers, const uint64_t* k, int32_t n_layers) {
  if (!layers || !k || n_layers < 1) return 0;
  size_t need = 0;
  for (int32_t i = 0; i < n_layers; ++i) {
    const size_t b = pvt_workspace_bytes(&layers[i], k[i]);
    if (b == 0) return 0;
    if (b > need) need = b;
  }
  return need;
}

int pvt_vstep_block(const pvt_layer* layers, const uint64_t* k, int32_t n_layers, uint32_t* const* idx_out,
                    void* const* W_hat, int32_t out_dtype, void* ws, size_t ws_bytes, void* cuda_stream) {
  if (!layers || !k || !idx_out || n_layers < 1) return PVT_EINVAL;
  // every layer is checked before anything is enqueued: the block is taken whole or not at all
  const size_t need = pvt_block_workspace_bytes(layers, k, n_layers);
  if (need == 0) {
    // find out which complaint it is: the per-layer calls below report it without launching (bad layers come first)
    for (int32_t i = 0; i < n_layers; ++i) {
      uint64_t G = 0;
      int rc = check_layer(&layers[i], &G);
      if (rc == PVT_OK) rc = check_quantiser(&layers[i]);
      if (rc != PVT_OK) return rc;
      if (k[i] < 1 || k[i] > G) return PVT_EINVAL;
    }
    return PVT_EINVAL;
  }
  if (ws_bytes < need) return PVT_EWORKSPACE;
  for (int32_t i = 0; i < n_layers; ++i) {
    const pvt_layer& L = layers[i];
    if (!idx_out[i] || !aligned4(idx_out[i]) || !L.W || !L.g || !L.scale || !L.codebooks || !L.codes) return PVT_EINVAL;
    if (!aligned16(L.W) || !aligned16(L.g) || !aligned16(L.codebooks) || !codes_aligned(&L)) return PVT_EINVAL;
    if (W_hat && W_hat[i] && !aligned16(W_hat[i])) return PVT_EINVAL;
  }
  if (W_hat && out_dtype != PVT_F32 && out_dtype != PVT_F16) return PVT_EINVAL;
  for (int32_t i = 0; i < n_layers; ++i) {
    int rc = pvt_vstep_select(&layers[i], k[i], idx_out[i], ws, ws_bytes, cuda_stream);
    if (rc == PVT_OK) rc = pvt_vstep_encode(&layers[i], idx_out[i], k[i], nullptr, ws, ws_bytes, cuda_stream);
    if (rc == PVT_OK && W_hat && W_hat[i]) rc = pvt_dequant(&layers[i], W_hat[i], out_dtype, nullptr, cuda_stream);
    if (rc != PVT_OK) return rc;
  }
  return PVT_OK;
}

int pvt_pstep_grad(const pvt_layer* layer, double* grad_codebooks, double* grad_scale, uint32_t* status,
                   void* cuda_stream) {
  uint64_t G = 0;
  int rc = check_layer(layer, &G);
  if (rc != PVT_OK) return rc;
  if ((rc = check_quantiser(layer)) != PVT_OK) return rc;
  if (!layer->g || !layer->scale || !layer->codebooks || !layer->codes || !grad_codebooks) return PVT_EINVAL;
  if (!aligned16(layer->g) || !aligned16(layer->codebooks)) return PVT_EINVAL;
  if ((reinterpret_cast<uintptr_t>(grad_codebooks) & 7u) || (reinterpret_cast<uintptr_t>(grad_scale) & 7u))
    return PVT_EINVAL;
  if (!codes_aligned(layer) || !aligned4(status)) return PVT_EINVAL;
  const cudaError_t e = launch_pstep_grad(*layer, G, grad_codebooks, grad_scale, status, sm_count(),
                                          static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? PVT_OK : fail_cuda(e);
}

int pvt_adam_update(float* param, void* param_f16, const double* grad, float* exp_avg, float* exp_avg_sq, uint64_t n,
                    float lr, float beta1, float beta2, float eps, float bias1, float bias2, void* cuda_stream) {
  if (!param || !grad || !exp_avg || !exp_avg_sq || n == 0) return PVT_EINVAL;
  if (!aligned4(param) || !aligned4(exp_avg) || !aligned4(exp_avg_sq) || (reinterpret_cast<uintptr_t>(grad) & 7u) ||
      (reinterpret_cast<uintptr_t>(param_f16) & 1u))
    return PVT_EINVAL;
  if (!(lr >= 0.0f) || !(beta1 >= 0.0f && beta1 < 1.0f) || !(beta2 >= 0.0f && beta2 < 1.0f) || !(eps >= 0.0f))
    return PVT_EINVAL;
  if (!(bias1 > 0.0f && bias1 <= 1.0f) || !(bias2 > 0.0f && bias2 <= 1.0f)) return PVT_EINVAL;
  const cudaError_t e = launch_adam(param, param_f16, grad, exp_avg, exp_avg_sq, n, lr, beta1, beta2, eps, bias1, bias2,
                                    sm_count(), static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? PVT_OK : fail_cuda(e);
}

int pvt_adam_direction(const float* grad, float* exp_avg, float* exp_avg_sq, float* dir, uint64_t n, float beta1,
                       float beta2, float eps, float bias1, float bias2, void* cuda_stream) {
  if (!grad || !exp_avg || !exp_avg_sq || !dir || n == 0 || n % 4 != 0) return PVT_EINVAL;
  if (!aligned16(grad) || !aligned16(exp_avg) || !aligned16(exp_avg_sq) || !aligned16(dir)) return PVT_EINVAL;
  if (!(beta1 >= 0.0f && beta1 < 1.0f) || !(beta2 >= 0.0f && beta2 < 1.0f) || !(eps >= 0.0f)) return PVT_EINVAL;
  if (!(bias1 > 0.0f && bias1 <= 1.0f) || !(bias2 > 0.0f && bias2 <= 1.0f)) return PVT_EINVAL;
  const cudaError_t e = launch_adam_direction(grad, exp_avg, exp_avg_sq, dir, n, beta1, beta2, eps, bias1, bias2,
                                              sm_count(), static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? PVT_OK : fail_cuda(e);
}

int pvt_status(void* ws, void* cuda_stream) {
  if (!ws) return PVT_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  uint32_t word = 0;
  cudaError_t e = cudaMemcpyAsync(&word, ws, sizeof(word), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e == cudaSuccess && word) e = cudaMemsetAsync(ws, 0, sizeof(word), s);
  if (e != cudaSuccess) return fail_cuda(e);
  return (int)(word & 0x7fffffffu);
}

const char* pvt_strerror(int code) {
  switch (code) {
    case PVT_OK: return "ok";
    case PVT_EINVAL: return "invalid argument (null or misaligned pointer, k out of range, bad shape or eta)";
    case PVT_EUNSUPPORTED: return "unsupported group_dim / codebook count / codebook size / dtype / beam";
    case PVT_EWORKSPACE: return "workspace smaller than pvt_workspace_bytes()";
    case PVT_ECUDA: return "CUDA runtime error (see pvt_last_cuda_error)";
    case PVT_ETOOLARGE: return "layer larger than the built-in scratch of pvt_vstep_select_noalloc (2^21 groups)";
    default: return code > 0 ? "device status bits set" : "unknown error";
  }
}

const char* pvt_last_cuda_error(void) { return cudaGetErrorString(g_last_cuda); }

int pvt_version(void) { return 100; }

void pvt_set_m1_search(int mode) {
  if (mode == PVT_M1_AUTO || mode == PVT_M1_FP32 || mode == PVT_M1_TENSOR) set_m1_search(mode);
}

unsigned long long pvt_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

void pvt_test_wait_limit(uint32_t max_polls, int64_t withhold_copy) {
  m1::set_wait_test_hook(max_polls == 0 ? m1::kMaxSpins : max_polls,
                         withhold_copy < 0 ? m1::kNoWithhold : (uint32_t)withhold_copy);
}

int pvt_adam_bias(uint64_t step, float beta1, float beta2, float* bias1_out, float* bias2_out) {
  if (step < 1 || !bias1_out || !bias2_out || !(beta1 >= 0.0f && beta1 < 1.0f) || !(beta2 >= 0.0f && beta2 < 1.0f))
    return PVT_EINVAL;
  // beta^t in binary64 from the binary32 beta widened exactly (the C library's pow), one rounding to binary32
  *bias1_out = (float)(1.0 - std::pow((double)beta1, (double)step));
  *bias2_out = (float)(1.0 - std::pow((double)beta2, (double)step));
  return PVT_OK;
}

int pvt_probe_fp32_tflops(float* scratch, size_t scratch_floats, float* tflops_out, void* cuda_stream) {
  if (!scratch || !tflops_out) return PVT_EINVAL;
  const int blocks = sm_count() * 8, iters = 8192;
  if (scratch_floats < (size_t)blocks * 256) return PVT_EWORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  cudaError_t e = cudaEventCreate(&e0);
  if (e == cudaSuccess) e = cudaEventCreate(&e1);
  if (e == cudaSuccess) {
    ffma_probe_kernel<<<blocks, 256, 0, s>>>(scratch, iters);  // warm-up
    cudaEventRecord(e0, s);
    ffma_probe_kernel<<<blocks, 256, 0, s>>>(scratch, iters);
    cudaEventRecord(e1, s);
    e = cudaEventSynchronize(e1);
  }
  float ms = 0.0f;
  if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  if (e != cudaSuccess) return fail_cuda(e);
  *tflops_out = (float)(2.0 * 16.0 * iters * 256.0 * blocks / (ms * 1e-3) / 1e12);
  return PVT_OK;
}

void pvt_timing_enable(int on) {
  Timing& t = timing();
  std::lock_guard<std::mutex> lock(t.mu);
  t.enabled = on != 0;
}

int pvt_timing_read(int kernel_id, float* total_ms, int* launches) {
  if (kernel_id < 0 || kernel_id >= kKernCount || !total_ms || !launches) return PVT_EINVAL;
  Timing& t = timing();
  std::lock_guard<std::mutex> lock(t.mu);
  float sum = 0.0f;
  int n = 0;
  for (auto& span : t.spans[kernel_id]) {
    float ms = 0.0f;
    cudaError_t e = cudaEventSynchronize(span.second);
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, span.first, span.second);
    cudaEventDestroy(span.first);
    cudaEventDestroy(span.second);
    if (e != cudaSuccess) {
      t.spans[kernel_id].clear();
      return fail_cuda(e);
    }
    sum += ms;
    ++n;
  }
  t.spans[kernel_id].clear();
  *total_ms = sum;
  *launches = n;
  return PVT_OK;
}

}  // extern "C"
