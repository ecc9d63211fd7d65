// C-ABI entry points: argument validation, workspace sizing, status handling.  Every step of the
// path runs in the CUDA kernels of route.cu / select.cu / prefill.cu; nothing here computes.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "common.cuh"

namespace crisp {

namespace {
thread_local char g_cuda_error[256] = "";

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}
}  // namespace

void set_cuda_error(cudaError_t e, const char* where) {
  std::snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", where, cudaGetErrorString(e));
}
void set_cu_error(const char* msg) { std::snprintf(g_cuda_error, sizeof(g_cuda_error), "%s", msg); }

int make_tmap_bf16_nhd(CUtensorMap* out, const void* base, int n, int heads, int box_rows) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) {
    set_cu_error("cuTensorMapEncodeTiled is not available (no CUDA driver?)");
    return CRISP_ERR_CUDA;
  }
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(kHeadDim), static_cast<cuuint64_t>(heads),
                              static_cast<cuuint64_t>(n)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(kHeadDim) * 2,
                                 static_cast<cuuint64_t>(heads) * kHeadDim * 2};
  const cuuint32_t box[3] = {64, 1, static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    char msg[96];
    std::snprintf(msg, sizeof(msg), "cuTensorMapEncodeTiled failed with CUresult %d", static_cast<int>(r));
    set_cu_error(msg);
    return CRISP_ERR_CUDA;
  }
  return CRISP_OK;
}

int validate(const crisp_params* p, Dims* d) {
  if (!p) return CRISP_ERR_INVALID_ARG;
  if (p->struct_size != static_cast<int32_t>(sizeof(crisp_params))) return CRISP_ERR_INVALID_ARG;
  if (p->seq_len <= 0 || p->n_q_heads <= 0 || p->n_kv_heads <= 0) return CRISP_ERR_INVALID_ARG;
  if (p->n_q_heads % p->n_kv_heads != 0) return CRISP_ERR_INVALID_ARG;
  if (p->sink_tokens < 1 || p->sink_tokens > p->seq_len) return CRISP_ERR_INVALID_ARG;
  if (p->local_tokens < 1 || p->local_tokens > p->seq_len) return CRISP_ERR_INVALID_ARG;
  if (p->k_min_blocks < 0) return CRISP_ERR_INVALID_ARG;
  if (p->selector < 0 || p->selector > 2) return CRISP_ERR_INVALID_ARG;
  if (p->force_pattern < 0 || p->force_pattern > 2) return CRISP_ERR_INVALID_ARG;
  if (!(p->alpha >= 0.f) || !(p->gamma > 0.f) || !std::isfinite(p->tau) || !std::isfinite(p->alpha) ||
      !std::isfinite(p->gamma) || !(p->softmax_scale >= 0.f) || !std::isfinite(p->softmax_scale))
    return CRISP_ERR_INVALID_ARG;
  if (p->head_dim != kHeadDim || p->block != kBlock) return CRISP_ERR_UNSUPPORTED;
  if (p->seq_len < 2 * kBlock) return CRISP_ERR_UNSUPPORTED;
  if (p->n_q_heads / p->n_kv_heads > kMaxGroup) return CRISP_ERR_UNSUPPORTED;
  if (p->seq_len > 8192 * kBlock) return CRISP_ERR_UNSUPPORTED;  // N_b limit of the selection kernels (1M tokens)
  d->n = p->seq_len;
  d->nb = (p->seq_len + kBlock - 1) / kBlock;
  d->nfull = p->seq_len / kBlock;
  d->rho = p->seq_len % kBlock;
  d->hq = p->n_q_heads;
  d->hkv = p->n_kv_heads;
  d->group = d->hq / d->hkv;
  d->w_sink = p->sink_tokens;
  d->w_local = p->local_tokens;
  d->n_sink_tiles = (d->w_sink + kBlock - 1) / kBlock;
  if (d->n_sink_tiles > d->nb) d->n_sink_tiles = d->nb;
  int fl = (d->n - d->w_local) / kBlock;
  d->first_local_tile = fl > d->n_sink_tiles ? fl : d->n_sink_tiles;
  d->n_anchor_slots = d->n_sink_tiles + (d->nb - d->first_local_tile);
  d->k_min = p->k_min_blocks;
  d->selector = p->selector;
  d->force_pattern = p->force_pattern;
  d->tau = p->tau;
  d->alpha = p->alpha;
  d->gamma = p->gamma;
  d->scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / std::sqrt(static_cast<float>(kHeadDim));
  d->scale_log2 = d->scale * kLog2e;
  return CRISP_OK;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace crisp

using namespace crisp;

extern "C" {

int crisp_version(void) { return 100; }

const char* crisp_status_string(int status) {
  switch (status) {
    case CRISP_OK: return "ok";
    case CRISP_ERR_INVALID_ARG: return "invalid argument";
    case CRISP_ERR_UNSUPPORTED: return "unsupported configuration";
    case CRISP_ERR_WORKSPACE: return "workspace too small or misaligned";
    case CRISP_ERR_CAPACITY: return "col_idx capacity too small";
    case CRISP_ERR_CUDA: return "CUDA error";
    case CRISP_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

const char* crisp_last_cuda_error(void) { return g_cuda_error; }

int crisp_workspace_bytes(const crisp_params* p, size_t* route_ws, size_t* select_ws, size_t* prefill_ws) {
  Dims d;
  int rc = validate(p, &d);
  if (rc != CRISP_OK) return rc;
  if (route_ws) *route_ws = route_ws_bytes(d);
  if (select_ws) *select_ws = select_ws_bytes(d);
  if (prefill_ws) *prefill_ws = prefill_ws_bytes(d);
  return CRISP_OK;
}

int crisp_route(const crisp_params* p, const void* q, const void* k, void* ws, size_t ws_bytes, float* c_struct,
                int32_t* pattern, float* p_v, float* p_s, void* cuda_stream) {
  Dims d;
  int rc = validate(p, &d);
  if (rc != CRISP_OK) return rc;
  if (!q || !k || !ws || !c_struct || !pattern || !p_v || !p_s) return CRISP_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k)) return CRISP_ERR_INVALID_ARG;
  if (!aligned16(ws) || ws_bytes < route_ws_bytes(d)) return CRISP_ERR_WORKSPACE;
  return launch_route(d, q, k, ws, c_struct, pattern, p_v, p_s, static_cast<cudaStream_t>(cuda_stream));
}

int crisp_route_static(const crisp_params* p, const void* q, const void* k, float* c_struct, int32_t* pattern,
                       float* p_v, float* p_s, int32_t* device_status, void* cuda_stream) {
  Dims d;
  int rc = validate(p, &d);
  if (rc != CRISP_OK) return rc;
  if (!q || !k || !c_struct || !pattern || !p_v || !p_s) return CRISP_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k)) return CRISP_ERR_INVALID_ARG;
  return launch_route_static(d, q, k, c_struct, pattern, p_v, p_s, device_status,
                             static_cast<cudaStream_t>(cuda_stream));
}

int crisp_select(const crisp_params* p, const void* q, const void* k, const int32_t* pattern, const float* p_v,
                 const float* p_s, void* ws, size_t ws_bytes, int64_t* row_ptr, int32_t* col_idx,
                 int64_t capacity, int64_t* nnz_needed, void* cuda_stream) {
  Dims d;
  int rc = validate(p, &d);
  if (rc != CRISP_OK) return rc;
  if (!q || !k || !pattern || !p_v || !p_s || !ws || !row_ptr || !nnz_needed) return CRISP_ERR_INVALID_ARG;
  if (capacity < 0 || (capacity > 0 && !col_idx)) return CRISP_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k)) return CRISP_ERR_INVALID_ARG;
  if (!aligned16(ws) || ws_bytes < select_ws_bytes(d)) return CRISP_ERR_WORKSPACE;
  return launch_select(d, q, k, pattern, p_v, p_s, ws, row_ptr, col_idx, capacity, nnz_needed,
                       static_cast<cudaStream_t>(cuda_stream));
}

int crisp_sparse_prefill(const crisp_params* p, const void* q, const void* k, const void* v,
                         const int64_t* row_ptr, const int32_t* col_idx, void* ws, size_t ws_bytes, void* o,
                         float* lse, void* cuda_stream) {
  Dims d;
  int rc = validate(p, &d);
  if (rc != CRISP_OK) return rc;
  if (!q || !k || !v || !row_ptr || !col_idx || !ws || !o) return CRISP_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return CRISP_ERR_INVALID_ARG;
  if (!aligned16(ws) || ws_bytes < prefill_ws_bytes(d)) return CRISP_ERR_WORKSPACE;
  return launch_prefill(d, q, k, v, row_ptr, col_idx, ws, o, lse, static_cast<cudaStream_t>(cuda_stream));
}

int crisp_dense_prefill(const crisp_params* p, const void* q, const void* k, const void* v, void* ws,
                        size_t ws_bytes, void* o, float* lse, void* cuda_stream) {
  Dims d;
  int rc = validate(p, &d);
  if (rc != CRISP_OK) return rc;
  if (!q || !k || !v || !ws || !o) return CRISP_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return CRISP_ERR_INVALID_ARG;
  if (!aligned16(ws) || ws_bytes < prefill_ws_bytes(d)) return CRISP_ERR_WORKSPACE;
  return launch_prefill(d, q, k, v, nullptr, nullptr, ws, o, lse, static_cast<cudaStream_t>(cuda_stream));
}

int crisp_route_jsd(const crisp_params* p, const void* q, const void* k, const float* p_v, void* select_ws,
                    size_t select_ws_bytes_, float tau_jsd, float* jsd, int32_t* pattern, void* cuda_stream) {
  Dims d;
  int rc = validate(p, &d);
  if (rc != CRISP_OK) return rc;
  if (!q || !k || !p_v || !select_ws || !jsd || !pattern) return CRISP_ERR_INVALID_ARG;
  if (!std::isfinite(tau_jsd)) return CRISP_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k)) return CRISP_ERR_INVALID_ARG;
  if (!aligned16(select_ws) || select_ws_bytes_ < select_ws_bytes(d)) return CRISP_ERR_WORKSPACE;
  return launch_route_jsd(d, q, k, p_v, select_ws, tau_jsd, jsd, pattern, static_cast<cudaStream_t>(cuda_stream));
}

int crisp_forward(const crisp_params* p, const void* q, const void* k, const void* v, void* route_ws,
                  size_t route_ws_bytes_, void* select_ws, size_t select_ws_bytes_, void* prefill_ws,
                  size_t prefill_ws_bytes_, float* c_struct, int32_t* pattern, float* p_v, float* p_s,
                  int64_t* row_ptr, int32_t* col_idx, int64_t capacity, int64_t* nnz_needed, void* o, float* lse,
                  int32_t dense_below_tokens, void* cuda_stream) {
  Dims d;
  int rc = validate(p, &d);
  if (rc != CRISP_OK) return rc;
  if (!q || !k || !v || !o || !prefill_ws) return CRISP_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return CRISP_ERR_INVALID_ARG;
  if (!aligned16(prefill_ws) || prefill_ws_bytes_ < prefill_ws_bytes(d)) return CRISP_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (d.n < dense_below_tokens) {
    // short prompt: routing and selection would cost more than they save
    return launch_prefill(d, q, k, v, nullptr, nullptr, prefill_ws, o, lse, st);
  }
  if (!route_ws || !select_ws || !c_struct || !pattern || !p_v || !p_s || !row_ptr || !nnz_needed)
    return CRISP_ERR_INVALID_ARG;
  if (capacity < 0 || (capacity > 0 && !col_idx)) return CRISP_ERR_INVALID_ARG;
  if (!aligned16(route_ws) || route_ws_bytes_ < route_ws_bytes(d)) return CRISP_ERR_WORKSPACE;
  if (!aligned16(select_ws) || select_ws_bytes_ < select_ws_bytes(d)) return CRISP_ERR_WORKSPACE;
  rc = launch_route(d, q, k, route_ws, c_struct, pattern, p_v, p_s, st);
  if (rc != CRISP_OK) return rc;
  rc = launch_select(d, q, k, pattern, p_v, p_s, select_ws, row_ptr, col_idx, capacity, nnz_needed, st);
  if (rc != CRISP_OK) return rc;
  // the status word of the selection stage gates the attention kernels: lists that did not fit are never read
  return launch_prefill(d, q, k, v, row_ptr, col_idx, prefill_ws, o, lse, st, static_cast<const int*>(select_ws));
}

int crisp_poll_device_status(void* ws, void* cuda_stream) {
  if (!ws) return CRISP_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int status = 0;
  CRISP_CUDA_TRY(cudaMemcpyAsync(&status, ws, sizeof(int), cudaMemcpyDeviceToHost, st), "poll: copy");
  CRISP_CUDA_TRY(cudaStreamSynchronize(st), "poll: synchronize");
  if (status != 0) CRISP_CUDA_TRY(cudaMemsetAsync(ws, 0, sizeof(int), st), "poll: clear");
  return status;
}

}  // extern "C"
