// Shared host/device declarations of the CRISP library internals (not part of the public ABI).
#pragma once
#include <cstddef>
#include <cstdint>
#include <utility>
#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include "../../include/crisp.h"

namespace crisp {

constexpr int kBlock = 128;       // B: tokens per block (Section 4.3)
constexpr int kHeadDim = 128;     // d
constexpr int kMaxGroup = 16;     // H_q / H_kv
constexpr size_t kWsHeader = 256; // bytes reserved at the start of every workspace (status word first)
constexpr float kLog2e = 1.4426950408889634f;

// Validated, derived problem sizes passed to kernels by value.
struct Dims {
  int n;          // seq_len
  int nb;         // N_b = ceil(n / B); the last block holds n - (N_b - 1) B tokens
  int nfull;      // floor(n / B)
  int rho;        // n mod B (0 when every block is full)
  int hq, hkv, group;
  int w_sink, w_local;
  int n_sink_tiles;    // key tiles intersecting [0, w_sink)
  int first_local_tile; // first key tile (>= n_sink_tiles) intersecting [n - w_local, n)
  int n_anchor_slots;  // n_sink_tiles + (nb - first_local_tile)
  int k_min, selector, force_pattern;
  float tau, alpha, gamma;
  float scale;      // softmax scale
  float scale_log2; // scale * log2(e)
};

int validate(const crisp_params* p, Dims* d, bool dense_only = false);
void set_cuda_error(cudaError_t e, const char* where);
void set_cu_error(const char* msg);

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Tensor map of a [n, H, 128] bf16 tensor with a {64, 1, 128} box and 128-byte swizzle.
int make_tmap_bf16_nhd(CUtensorMap* out, const void* base, int n, int heads, int box_rows = 128);

#define CRISP_CUDA_TRY(expr, where)              \
  do {                                           \
    cudaError_t e__ = (expr);                    \
    if (e__ != cudaSuccess) {                    \
      ::crisp::set_cuda_error(e__, where);       \
      return CRISP_ERR_CUDA;                     \
    }                                            \
  } while (0)

// Optional per-kernel timing (diagnostic, off by default; see crisp_profile_enable): while it is on, every kernel
// launch of the stage launchers is bracketed by a pair of CUDA events on the caller's stream.
bool prof_enabled();
void prof_begin(const char* name, cudaStream_t stream);
void prof_end(cudaStream_t stream);
struct ProfScope {
  cudaStream_t stream;
  bool on;
  ProfScope(const char* name, cudaStream_t s) : stream(s), on(prof_enabled()) {
    if (on) prof_begin(name, stream);
  }
  ~ProfScope() {
    if (on) prof_end(stream);
  }
};
// CRISP_KERNEL("name", stream, launch_pdl(kernel, grid, block, smem, stream, args...));
#define CRISP_KERNEL(name, stream, ...)          \
  do {                                           \
    ::crisp::ProfScope prof_scope__(name, stream); \
    __VA_ARGS__;                                 \
  } while (0)

#ifdef __CUDACC__
// Launch with programmatic dependent launch allowed: the kernel's CTAs may become resident while the kernel
// before it on the stream is still running.  Every kernel launched this way calls pdl_enter() as its first
// statement, which lets the kernel after it do the same and then waits until the kernel before it has
// completed and its writes are visible, so the stream's order is kept; what is saved is the launch latency
// between two short kernels.  (A kernel that follows a memset or an event record simply starts after it.)
template <typename... KArgs, typename... Args>
inline void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                       Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr = {};
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(std::forward<Args>(args))...);  // errors: cudaGetLastError
}
__device__ __forceinline__ void pdl_enter() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
#endif

#ifdef __CUDACC__
// Exclusive prefix sum over the kThreads threads of a block (a multiple of 32, at most 1024), in thread order
// (warp shuffles, then the warp totals).  `scratch` holds 33 values; `*total` (optional) receives the sum of all
// threads.  Every thread of the block must call it; it contains three __syncthreads and leaves `scratch` reusable
// after the last.
template <int kThreads>
__device__ __forceinline__ long long block_exclusive_scan(long long v, long long* scratch, long long* total) {
  constexpr int kWarps = kThreads / 32;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  long long incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const long long t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  __syncthreads();  // scratch may still be read from a previous call
  if (lane == 31) scratch[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const long long wt = lane < kWarps ? scratch[lane] : 0;
    long long wi = wt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const long long t = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += t;
    }
    if (lane < kWarps) scratch[lane] = wi - wt;
    if (lane == 31) scratch[32] = wi;
  }
  __syncthreads();
  if (total) *total = scratch[32];
  return scratch[warp] + (incl - v);
}
__device__ __forceinline__ long long block_exclusive_scan_1024(long long v, long long* scratch, long long* total) {
  return block_exclusive_scan<1024>(v, scratch, total);
}
#endif

// stage launchers (each enqueues on `stream` and returns a crisp_status)
int launch_route(const Dims& d, const void* q, const void* k, void* ws, float* c_struct, int32_t* pattern,
                 float* p_v, float* p_s, cudaStream_t stream);
size_t route_ws_bytes(const Dims& d);
int launch_route_static(const Dims& d, const void* q, const void* k, float* c_struct, int32_t* pattern,
                        float* p_v, float* p_s, int32_t* device_status, cudaStream_t stream);
int launch_select(const Dims& d, const void* q, const void* k, const int32_t* pattern, const float* p_v,
                  const float* p_s, void* ws, int64_t* row_ptr, int32_t* col_idx, int64_t capacity,
                  int64_t* nnz_needed, cudaStream_t stream);
size_t select_ws_bytes(const Dims& d);
int launch_route_jsd(const Dims& d, const void* q, const void* k, const float* p_v, void* ws, float tau_jsd,
                     float* jsd, int32_t* pattern, cudaStream_t stream);
int launch_prefill(const Dims& d, const void* q, const void* k, const void* v, const int64_t* row_ptr,
                   const int32_t* col_idx, void* ws, void* o, float* lse, cudaStream_t stream,
                   const int* gate = nullptr);
size_t prefill_ws_bytes(const Dims& d);
int launch_selftest_bounded_wait(void* ws, long long limit_ns, cudaStream_t stream);

}  // namespace crisp
