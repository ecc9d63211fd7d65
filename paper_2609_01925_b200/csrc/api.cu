// C-ABI entry points: argument validation, workspace sizing, status handling.  Every step of the
// path runs in the CUDA kernels of route.cu / select.cu / prefill.cu; nothing here computes.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <vector>

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

// ---- optional per-kernel timing
namespace {
struct ProfRecord {
  const char* name;
  cudaEvent_t begin, end;
};
std::mutex g_prof_mutex;
bool g_prof_on = false;
std::vector<ProfRecord> g_prof_records;
std::vector<cudaEvent_t> g_prof_free;  // events of earlier records, reused

cudaEvent_t prof_event() {
  if (!g_prof_free.empty()) {
    cudaEvent_t e = g_prof_free.back();
    g_prof_free.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
  return e;
}
}  // namespace

bool prof_enabled() {
  std::lock_guard<std::mutex> lock(g_prof_mutex);
  return g_prof_on;
}
void prof_begin(const char* name, cudaStream_t stream) {
  std::lock_guard<std::mutex> lock(g_prof_mutex);
  if (!g_prof_on) return;
  ProfRecord r{name, prof_event(), prof_event()};
  if (r.begin) cudaEventRecord(r.begin, stream);
  g_prof_records.push_back(r);
}
void prof_end(cudaStream_t stream) {
  std::lock_guard<std::mutex> lock(g_prof_mutex);
  if (!g_prof_on || g_prof_records.empty()) return;
  ProfRecord& r = g_prof_records.back();
  if (r.end) cudaEventRecord(r.end, stream);
}

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

// dense_only: the call runs dense attention alone, which is defined for every length >= 1 and reads none of
// the routing parameters' relation to the length.
int validate(const crisp_params* p, Dims* d, bool dense_only) {
  if (!p) return CRISP_ERR_INVALID_ARG;
  if (p->struct_size != static_cast<int32_t>(sizeof(crisp_params))) return CRISP_ERR_INVALID_ARG;
  if (p->seq_len <= 0 || p->n_q_heads <= 0 || p->n_kv_heads <= 0) return CRISP_ERR_INVALID_ARG;
  if (p->n_q_heads % p->n_kv_heads != 0) return CRISP_ERR_INVALID_ARG;
  // fewer than two blocks cannot be routed; said before the windows are compared with the length
  if (!dense_only && p->seq_len < 2 * kBlock && p->head_dim == kHeadDim && p->block == kBlock)
    return CRISP_ERR_UNSUPPORTED;
  if (p->sink_tokens < 1 || (!dense_only && p->sink_tokens > p->seq_len)) return CRISP_ERR_INVALID_ARG;
  if (p->local_tokens < 1 || (!dense_only && p->local_tokens > p->seq_len)) return CRISP_ERR_INVALID_ARG;
  if (p->k_min_blocks < 0) return CRISP_ERR_INVALID_ARG;
  if (p->selector < 0 || p->selector > 2) return CRISP_ERR_INVALID_ARG;
  if (p->force_pattern < 0 || p->force_pattern > 2) return CRISP_ERR_INVALID_ARG;
  if (!(p->alpha >= 0.f) || !(p->gamma > 0.f) || !std::isfinite(p->tau) || !std::isfinite(p->alpha) ||
      !std::isfinite(p->gamma) || !(p->softmax_scale >= 0.f) || !std::isfinite(p->softmax_scale))
    return CRISP_ERR_INVALID_ARG;
  if (p->head_dim != kHeadDim || p->block != kBlock) return CRISP_ERR_UNSUPPORTED;
  if (!dense_only && p->seq_len < 2 * kBlock) return CRISP_ERR_UNSUPPORTED;
  if (p->n_q_heads / p->n_kv_heads > kMaxGroup) return CRISP_ERR_UNSUPPORTED;
  if (p->seq_len > 8192 * kBlock) return CRISP_ERR_UNSUPPORTED;  // N_b limit of the selection kernels (1M tokens)
  d->n = p->seq_len;
  d->nb = (p->seq_len + kBlock - 1) / kBlock;
  d->nfull = p->seq_len / kBlock;
  d->rho = p->seq_len % kBlock;
  d->hq = p->n_q_heads;
  d->hkv = p->n_kv_heads;
  d->group = d->hq / d->hkv;
  d->w_sink = p->sink_tokens < p->seq_len ? p->sink_tokens : p->seq_len;
  d->w_local = p->local_tokens < p->seq_len ? p->local_tokens : p->seq_len;
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
    case CRISP_ERR_BAD_LIST: return "index lists break the list rules";
    default: return "unknown status";
  }
}

const char* crisp_last_cuda_error(void) { return g_cuda_error; }

int crisp_workspace_bytes(const crisp_params* p, size_t* route_ws, size_t* select_ws, size_t* prefill_ws) {
  Dims d;
  if (p && p->seq_len > 0 && p->seq_len < 2 * kBlock) {
    // too short to be routed: only dense attention applies, and only its workspace is needed
    const int rc_dense = validate(p, &d, /*dense_only=*/true);
    if (rc_dense != CRISP_OK) return rc_dense;
    if (route_ws) *route_ws = 0;
    if (select_ws) *select_ws = 0;
    if (prefill_ws) *prefill_ws = prefill_ws_bytes(d);
    return CRISP_OK;
  }
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
  int rc = validate(p, &d, /*dense_only=*/true);
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
  const bool gated = p && p->seq_len < dense_below_tokens;
  int rc = validate(p, &d, gated);
  if (rc != CRISP_OK) return rc;
  if (!q || !k || !v || !o || !prefill_ws) return CRISP_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return CRISP_ERR_INVALID_ARG;
  if (!aligned16(prefill_ws) || prefill_ws_bytes_ < prefill_ws_bytes(d)) return CRISP_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (gated) {
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

namespace {
// Is sequence length `len` of a packed batch routed (true) or sent to dense attention (false)?
bool varlen_routed(int64_t len, int32_t dense_below_tokens) {
  return len >= 2 * kBlock && len >= dense_below_tokens;
}
}  // namespace

int crisp_varlen_layout(const crisp_params* p, const int64_t* cu_seqlens, int32_t batch, int64_t capacity,
                        int32_t dense_below_tokens, int64_t* blk_off, int64_t* col_off) {
  if (!p || !cu_seqlens || batch < 0 || capacity < 0 || !blk_off || !col_off) return CRISP_ERR_INVALID_ARG;
  if (p->n_q_heads <= 0) return CRISP_ERR_INVALID_ARG;
  if (cu_seqlens[0] != 0) return CRISP_ERR_INVALID_ARG;
  // causal blocks of the routed sequences: the shares of col_idx
  unsigned __int128 total = 0;
  blk_off[0] = 0;
  for (int b = 0; b < batch; ++b) {
    const int64_t len = cu_seqlens[b + 1] - cu_seqlens[b];
    if (len < 0 || len > 8192LL * kBlock) return len < 0 ? CRISP_ERR_INVALID_ARG : CRISP_ERR_UNSUPPORTED;
    const int64_t nb = (len + kBlock - 1) / kBlock;
    blk_off[b + 1] = blk_off[b] + nb;
    if (varlen_routed(len, dense_below_tokens)) total += static_cast<unsigned __int128>(nb) * (nb + 1) / 2;
  }
  unsigned __int128 run = 0;
  col_off[0] = 0;
  for (int b = 0; b < batch; ++b) {
    const int64_t len = cu_seqlens[b + 1] - cu_seqlens[b];
    const int64_t nb = (len + kBlock - 1) / kBlock;
    if (varlen_routed(len, dense_below_tokens)) run += static_cast<unsigned __int128>(nb) * (nb + 1) / 2;
    col_off[b + 1] = total == 0 ? 0 : static_cast<int64_t>(static_cast<unsigned __int128>(capacity) * run / total);
  }
  return CRISP_OK;
}

int crisp_forward_varlen(const crisp_params* p, const int64_t* cu_seqlens, int32_t batch, const void* q, const void* k,
                         const void* v, void* route_ws, size_t route_ws_bytes_, void* select_ws,
                         size_t select_ws_bytes_, void* prefill_ws, size_t prefill_ws_bytes_, float* c_struct,
                         int32_t* pattern, float* p_v, float* p_s, int64_t* row_ptr, int32_t* col_idx, int64_t capacity,
                         int64_t* nnz_needed, int32_t* device_status, void* o, float* lse, int32_t dense_below_tokens,
                         void* cuda_stream) {
  if (!p || !cu_seqlens || batch < 0) return CRISP_ERR_INVALID_ARG;
  if (p->struct_size != static_cast<int32_t>(sizeof(crisp_params))) return CRISP_ERR_INVALID_ARG;
  if (batch == 0) return CRISP_OK;
  if (!q || !k || !v || !o || !prefill_ws) return CRISP_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return CRISP_ERR_INVALID_ARG;
  if (capacity < 0 || (capacity > 0 && !col_idx)) return CRISP_ERR_INVALID_ARG;
  std::vector<int64_t> blk_off, col_off;
  std::vector<Dims> dims;
  try {
    blk_off.resize(static_cast<size_t>(batch) + 1);
    col_off.resize(static_cast<size_t>(batch) + 1);
    dims.resize(static_cast<size_t>(batch));
  } catch (...) {
    return CRISP_ERR_INVALID_ARG;  // a batch too large to describe on the host
  }
  int rc = crisp_varlen_layout(p, cu_seqlens, batch, capacity, dense_below_tokens, blk_off.data(), col_off.data());
  if (rc != CRISP_OK) return rc;

  // ---- first pass: every sequence's parameters and workspace needs, before anything is enqueued
  bool any_routed = false;
  for (int b = 0; b < batch; ++b) {
    const int64_t len = cu_seqlens[b + 1] - cu_seqlens[b];
    if (len == 0) continue;
    crisp_params pb = *p;
    pb.seq_len = static_cast<int32_t>(len);
    const bool routed = varlen_routed(len, dense_below_tokens);
    rc = validate(&pb, &dims[b], !routed);
    if (rc != CRISP_OK) return rc;
    if (!aligned16(prefill_ws) || prefill_ws_bytes_ < prefill_ws_bytes(dims[b])) return CRISP_ERR_WORKSPACE;
    if (routed) {
      any_routed = true;
      if (!route_ws || !select_ws) return CRISP_ERR_INVALID_ARG;
      if (!aligned16(route_ws) || route_ws_bytes_ < route_ws_bytes(dims[b])) return CRISP_ERR_WORKSPACE;
      if (!aligned16(select_ws) || select_ws_bytes_ < select_ws_bytes(dims[b])) return CRISP_ERR_WORKSPACE;
    }
  }
  if (any_routed && (!c_struct || !pattern || !p_v || !p_s || !row_ptr || !nnz_needed)) return CRISP_ERR_INVALID_ARG;

  // ---- second pass: one sequence after the other on the stream; the workspaces are reused in stream order
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t hq = static_cast<size_t>(p->n_q_heads), hkv = static_cast<size_t>(p->n_kv_heads);
  for (int b = 0; b < batch; ++b) {
    const int64_t t0 = cu_seqlens[b], len = cu_seqlens[b + 1] - t0;
    if (device_status)
      CRISP_CUDA_TRY(cudaMemsetAsync(device_status + 2 * b, 0, 2 * sizeof(int32_t), st), "forward_varlen: clear status");
    if (len == 0) continue;
    const Dims& d = dims[b];
    const char* qb = static_cast<const char*>(q) + static_cast<size_t>(t0) * hq * kHeadDim * 2;
    const char* kb = static_cast<const char*>(k) + static_cast<size_t>(t0) * hkv * kHeadDim * 2;
    const char* vb = static_cast<const char*>(v) + static_cast<size_t>(t0) * hkv * kHeadDim * 2;
    char* ob = static_cast<char*>(o) + static_cast<size_t>(t0) * hq * kHeadDim * 2;
    float* lb = lse ? lse + static_cast<size_t>(t0) * hq : nullptr;
    if (!varlen_routed(len, dense_below_tokens)) {
      rc = launch_prefill(d, qb, kb, vb, nullptr, nullptr, prefill_ws, ob, lb, st);
      if (rc != CRISP_OK) return rc;
    } else {
      float* cs = c_struct + static_cast<size_t>(b) * hq;
      int32_t* pat = pattern + static_cast<size_t>(b) * hq;
      float* pv = p_v + static_cast<size_t>(blk_off[b]) * hq;
      float* ps = p_s + static_cast<size_t>(blk_off[b]) * hq;
      int64_t* rp = row_ptr + (static_cast<size_t>(blk_off[b]) + b) * hq;
      int32_t* ci = col_idx ? col_idx + col_off[b] : nullptr;
      const int64_t cap = col_off[b + 1] - col_off[b];
      rc = launch_route(d, qb, kb, route_ws, cs, pat, pv, ps, st);
      if (rc != CRISP_OK) return rc;
      rc = launch_select(d, qb, kb, pat, pv, ps, select_ws, rp, ci, cap, nnz_needed + b, st);
      if (rc != CRISP_OK) return rc;
      rc = launch_prefill(d, qb, kb, vb, rp, ci, prefill_ws, ob, lb, st, static_cast<const int*>(select_ws));
      if (rc != CRISP_OK) return rc;
      if (device_status)
        CRISP_CUDA_TRY(cudaMemcpyAsync(device_status + 2 * b, select_ws, sizeof(int32_t), cudaMemcpyDeviceToDevice, st),
                       "forward_varlen: selection status");
    }
    if (device_status)
      CRISP_CUDA_TRY(cudaMemcpyAsync(device_status + 2 * b + 1, prefill_ws, sizeof(int32_t), cudaMemcpyDeviceToDevice, st),
                     "forward_varlen: attention status");
  }
  return CRISP_OK;
}

int crisp_profile_enable(int on) {
  std::lock_guard<std::mutex> lock(g_prof_mutex);
  for (ProfRecord& r : g_prof_records) {
    if (r.begin) g_prof_free.push_back(r.begin);
    if (r.end) g_prof_free.push_back(r.end);
  }
  g_prof_records.clear();
  g_prof_on = on != 0;
  return CRISP_OK;
}

int crisp_profile_read(char* names, size_t names_bytes, float* ms, int32_t max_records, int32_t* n_records) {
  if (!n_records || max_records < 0 || (max_records > 0 && (!names || !ms))) return CRISP_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_prof_mutex);
  size_t used = 0;
  int32_t n = 0;
  if (names && names_bytes > 0) names[0] = 0;
  for (const ProfRecord& r : g_prof_records) {
    if (n >= max_records) break;
    const size_t len = std::strlen(r.name);
    if (used + len + 2 > names_bytes) break;
    float t = -1.f;
    if (r.begin && r.end) {
      CRISP_CUDA_TRY(cudaEventSynchronize(r.end), "profile: synchronize");
      CRISP_CUDA_TRY(cudaEventElapsedTime(&t, r.begin, r.end), "profile: elapsed time");
    }
    std::memcpy(names + used, r.name, len);
    used += len;
    names[used++] = '\n';
    names[used] = 0;
    ms[n++] = t;
  }
  *n_records = n;
  return CRISP_OK;
}

int crisp_selftest_bounded_wait(void* ws, size_t ws_bytes, int64_t limit_ns, void* cuda_stream) {
  if (!ws) return CRISP_ERR_INVALID_ARG;
  if (!aligned16(ws) || ws_bytes < kWsHeader) return CRISP_ERR_WORKSPACE;
  return launch_selftest_bounded_wait(ws, limit_ns, static_cast<cudaStream_t>(cuda_stream));
}

namespace {
// Carving of crisp_forward_host's staging buffer for one chunk shape.
struct HostStage {
  void* q[2];
  void* k[2];
  void* v[2];
  void* o[2];
  void* route_ws;
  void* select_ws;
  void* prefill_ws;
  float* c_struct;
  int32_t* pattern;
  float* p_v;
  float* p_s;
  int64_t* row_ptr;
  int64_t* nnz;
  int32_t* col_idx;
  int64_t capacity;
  size_t route_bytes, select_bytes, prefill_bytes;
};
HostStage carve_host_stage(const Dims& dc, void* stage, size_t* total) {
  HostStage hs;
  uint8_t* base = static_cast<uint8_t*>(stage);
  size_t off = 0;
  auto take = [&](size_t bytes) {
    void* ptr = base + off;
    off += (bytes + 255) & ~static_cast<size_t>(255);
    return ptr;
  };
  const size_t qo = static_cast<size_t>(dc.n) * dc.hq * kHeadDim * 2, kv = static_cast<size_t>(dc.n) * dc.hkv * kHeadDim * 2;
  for (int b = 0; b < 2; ++b) {
    hs.q[b] = take(qo);
    hs.k[b] = take(kv);
    hs.v[b] = take(kv);
    hs.o[b] = take(qo);
  }
  hs.route_bytes = route_ws_bytes(dc);
  hs.select_bytes = select_ws_bytes(dc);
  hs.prefill_bytes = prefill_ws_bytes(dc);
  hs.route_ws = take(hs.route_bytes);
  hs.select_ws = take(hs.select_bytes);
  hs.prefill_ws = take(hs.prefill_bytes);
  hs.c_struct = static_cast<float*>(take(sizeof(float) * dc.hq));
  hs.pattern = static_cast<int32_t*>(take(sizeof(int32_t) * dc.hq));
  hs.p_v = static_cast<float*>(take(sizeof(float) * dc.hq * dc.nb));
  hs.p_s = static_cast<float*>(take(sizeof(float) * dc.hq * dc.nb));
  hs.row_ptr = static_cast<int64_t*>(take(sizeof(int64_t) * dc.hq * (dc.nb + 1)));
  hs.nnz = static_cast<int64_t*>(take(sizeof(int64_t)));
  hs.capacity = static_cast<int64_t>(dc.hq) * dc.nb * (static_cast<int64_t>(dc.nb) + 1) / 2;
  hs.col_idx = static_cast<int32_t*>(take(sizeof(int32_t) * static_cast<size_t>(hs.capacity)));
  *total = off;
  return hs;
}
// chunk shape: the layer's parameters with kv_groups_per_chunk KV groups
int chunk_dims(const crisp_params* p, int32_t gpc, crisp_params* pc, Dims* dc) {
  Dims d;
  int rc = validate(p, &d);
  if (rc != CRISP_OK) return rc;
  if (gpc < 1 || gpc > p->n_kv_heads || p->n_kv_heads % gpc != 0) return CRISP_ERR_INVALID_ARG;
  *pc = *p;
  pc->n_kv_heads = gpc;
  pc->n_q_heads = gpc * (p->n_q_heads / p->n_kv_heads);
  return validate(pc, dc);
}
// copy streams of crisp_forward_host and a page-locked block for the per-chunk status words, per device
struct HostPipe {
  cudaStream_t in = nullptr, out = nullptr;
  int* words = nullptr;  // [kMaxChunks][8]: three status words, nnz (two words)
  std::mutex busy;       // one crisp_forward_host call per device at a time (they share the block above)
};
constexpr int kMaxChunks = 1024;
std::mutex g_pipe_mutex;
HostPipe g_pipes[64];
int host_pipe(HostPipe** out) {
  int dev = 0;
  CRISP_CUDA_TRY(cudaGetDevice(&dev), "forward_host: device");
  if (dev < 0 || dev >= 64) return CRISP_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  HostPipe& hp = g_pipes[dev];
  if (!hp.in) CRISP_CUDA_TRY(cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking), "forward_host: stream");
  if (!hp.out) CRISP_CUDA_TRY(cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking), "forward_host: stream");
  if (!hp.words) CRISP_CUDA_TRY(cudaHostAlloc(&hp.words, sizeof(int) * 8 * kMaxChunks, cudaHostAllocDefault), "forward_host: status block");
  *out = &hp;
  return CRISP_OK;
}
}  // namespace

size_t crisp_forward_host_stage_bytes(const crisp_params* p, int32_t kv_groups_per_chunk) {
  crisp_params pc;
  Dims dc;
  if (chunk_dims(p, kv_groups_per_chunk, &pc, &dc) != CRISP_OK) return 0;
  size_t total = 0;
  carve_host_stage(dc, nullptr, &total);
  return total;
}

int crisp_forward_host(const crisp_params* p, const void* q_host, const void* k_host, const void* v_host,
                       void* o_host, int32_t kv_groups_per_chunk, void* stage, size_t stage_bytes,
                       int32_t* pattern_host, int64_t* nnz_host, void* cuda_stream) {
  crisp_params pc;
  Dims dc;
  int rc = chunk_dims(p, kv_groups_per_chunk, &pc, &dc);
  if (rc != CRISP_OK) return rc;
  if (!q_host || !k_host || !v_host || !o_host || !stage) return CRISP_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(stage) & 255) != 0) return CRISP_ERR_WORKSPACE;
  size_t need = 0;
  const HostStage hs = carve_host_stage(dc, stage, &need);
  if (stage_bytes < need) return CRISP_ERR_WORKSPACE;
  const int n_chunks = p->n_kv_heads / kv_groups_per_chunk;
  if (n_chunks > kMaxChunks) return CRISP_ERR_UNSUPPORTED;
  HostPipe* hp = nullptr;
  rc = host_pipe(&hp);
  if (rc != CRISP_OK) return rc;
  std::lock_guard<std::mutex> one_call(hp->busy);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

  // events: [buffer] inputs on the device / kernels finished / output on the host
  cudaEvent_t in_done[2] = {nullptr, nullptr}, comp_done[2] = {nullptr, nullptr}, out_done[2] = {nullptr, nullptr};
  cudaEvent_t start = nullptr;
  auto destroy = [&]() {
    for (int b = 0; b < 2; ++b) {
      if (in_done[b]) cudaEventDestroy(in_done[b]);
      if (comp_done[b]) cudaEventDestroy(comp_done[b]);
      if (out_done[b]) cudaEventDestroy(out_done[b]);
    }
    if (start) cudaEventDestroy(start);
  };
  cudaError_t ce = cudaEventCreateWithFlags(&start, cudaEventDisableTiming);
  for (int b = 0; b < 2 && ce == cudaSuccess; ++b) {
    ce = cudaEventCreateWithFlags(&in_done[b], cudaEventDisableTiming);
    if (ce == cudaSuccess) ce = cudaEventCreateWithFlags(&comp_done[b], cudaEventDisableTiming);
    if (ce == cudaSuccess) ce = cudaEventCreateWithFlags(&out_done[b], cudaEventDisableTiming);
  }
  if (ce != cudaSuccess) {
    destroy();
    set_cuda_error(ce, "forward_host: events");
    return CRISP_ERR_CUDA;
  }
#define CRISP_FH_TRY(expr, where)        \
  do {                                   \
    cudaError_t e__ = (expr);            \
    if (e__ != cudaSuccess) {            \
      cudaStreamSynchronize(hp->in);     \
      cudaStreamSynchronize(st);         \
      cudaStreamSynchronize(hp->out);    \
      destroy();                         \
      set_cuda_error(e__, where);        \
      return CRISP_ERR_CUDA;             \
    }                                    \
  } while (0)

  // the copy streams start behind whatever the caller has already enqueued on cuda_stream
  CRISP_FH_TRY(cudaEventRecord(start, st), "forward_host: record");
  CRISP_FH_TRY(cudaStreamWaitEvent(hp->in, start, 0), "forward_host: wait");
  CRISP_FH_TRY(cudaStreamWaitEvent(hp->out, start, 0), "forward_host: wait");
  const size_t row_q = static_cast<size_t>(p->n_q_heads) * kHeadDim * 2, row_kv = static_cast<size_t>(p->n_kv_heads) * kHeadDim * 2;
  const size_t row_qc = static_cast<size_t>(dc.hq) * kHeadDim * 2, row_kvc = static_cast<size_t>(dc.hkv) * kHeadDim * 2;
  int launch_rc = CRISP_OK;
  for (int c = 0; c < n_chunks && launch_rc == CRISP_OK; ++c) {
    const int b = c & 1;
    // ---- inputs of chunk c: its heads are a column slice of every token's row
    if (c >= 2) CRISP_FH_TRY(cudaStreamWaitEvent(hp->in, comp_done[b], 0), "forward_host: wait");  // chunk c - 2 has read buffer b
    CRISP_FH_TRY(cudaMemcpy2DAsync(hs.k[b], row_kvc, static_cast<const uint8_t*>(k_host) + c * row_kvc, row_kv, row_kvc, dc.n,
                                   cudaMemcpyHostToDevice, hp->in), "forward_host: copy K");
    CRISP_FH_TRY(cudaMemcpy2DAsync(hs.q[b], row_qc, static_cast<const uint8_t*>(q_host) + c * row_qc, row_q, row_qc, dc.n,
                                   cudaMemcpyHostToDevice, hp->in), "forward_host: copy Q");
    CRISP_FH_TRY(cudaMemcpy2DAsync(hs.v[b], row_kvc, static_cast<const uint8_t*>(v_host) + c * row_kvc, row_kv, row_kvc, dc.n,
                                   cudaMemcpyHostToDevice, hp->in), "forward_host: copy V");
    CRISP_FH_TRY(cudaEventRecord(in_done[b], hp->in), "forward_host: record");
    // ---- kernels of chunk c
    CRISP_FH_TRY(cudaStreamWaitEvent(st, in_done[b], 0), "forward_host: wait");
    if (c >= 2) CRISP_FH_TRY(cudaStreamWaitEvent(st, out_done[b], 0), "forward_host: wait");  // O of chunk c - 2 has left buffer b
    launch_rc = crisp_forward(&pc, hs.q[b], hs.k[b], hs.v[b], hs.route_ws, hs.route_bytes, hs.select_ws, hs.select_bytes,
                              hs.prefill_ws, hs.prefill_bytes, hs.c_struct, hs.pattern, hs.p_v, hs.p_s, hs.row_ptr,
                              hs.col_idx, hs.capacity, hs.nnz, hs.o[b], nullptr, 0, st);
    if (launch_rc != CRISP_OK) break;
    // the chunk's status words, list size and labels leave on the kernels' stream, before the next chunk reuses them
    int* wd = hp->words + 8 * c;
    CRISP_FH_TRY(cudaMemcpyAsync(wd + 0, hs.route_ws, sizeof(int), cudaMemcpyDeviceToHost, st), "forward_host: status");
    CRISP_FH_TRY(cudaMemcpyAsync(wd + 1, hs.select_ws, sizeof(int), cudaMemcpyDeviceToHost, st), "forward_host: status");
    CRISP_FH_TRY(cudaMemcpyAsync(wd + 2, hs.prefill_ws, sizeof(int), cudaMemcpyDeviceToHost, st), "forward_host: status");
    CRISP_FH_TRY(cudaMemcpyAsync(wd + 4, hs.nnz, sizeof(int64_t), cudaMemcpyDeviceToHost, st), "forward_host: nnz");
    if (pattern_host)
      CRISP_FH_TRY(cudaMemcpyAsync(pattern_host + c * dc.hq, hs.pattern, sizeof(int32_t) * dc.hq, cudaMemcpyDeviceToHost, st),
                   "forward_host: labels");
    CRISP_FH_TRY(cudaEventRecord(comp_done[b], st), "forward_host: record");
    // ---- output of chunk c
    CRISP_FH_TRY(cudaStreamWaitEvent(hp->out, comp_done[b], 0), "forward_host: wait");
    CRISP_FH_TRY(cudaMemcpy2DAsync(static_cast<uint8_t*>(o_host) + c * row_qc, row_q, hs.o[b], row_qc, row_qc, dc.n,
                                   cudaMemcpyDeviceToHost, hp->out), "forward_host: copy O");
    CRISP_FH_TRY(cudaEventRecord(out_done[b], hp->out), "forward_host: record");
  }
  // everything this call enqueued has finished when the three streams are idle; cuda_stream also waits for the
  // last output copy, so work the caller enqueues behind this call sees o_host complete
  cudaError_t e_in = cudaStreamSynchronize(hp->in), e_st = cudaStreamSynchronize(st), e_out = cudaStreamSynchronize(hp->out);
  destroy();
#undef CRISP_FH_TRY
  if (launch_rc != CRISP_OK) return launch_rc;
  if (e_in != cudaSuccess || e_st != cudaSuccess || e_out != cudaSuccess) {
    set_cuda_error(e_in != cudaSuccess ? e_in : (e_st != cudaSuccess ? e_st : e_out), "forward_host: synchronize");
    return CRISP_ERR_CUDA;
  }
  int64_t nnz = 0;
  for (int c = 0; c < n_chunks; ++c) {
    const int* wd = hp->words + 8 * c;
    for (int i = 0; i < 3; ++i)
      if (wd[i] != 0) return wd[i];
    int64_t chunk_nnz;
    std::memcpy(&chunk_nnz, wd + 4, sizeof(chunk_nnz));
    nnz += chunk_nnz;
  }
  if (nnz_host) *nnz_host = nnz;
  return CRISP_OK;
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
