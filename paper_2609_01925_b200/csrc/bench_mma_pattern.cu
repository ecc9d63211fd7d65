// Stand-alone micro-benchmark of the attention kernel's MMA issue pattern in isolation: one thread per CTA issues
// 8 SS MMAs (S = Q K^T, both operands in shared memory) and 8 TS MMAs (O += P V, A in TMEM) per step, optionally
// with the commits and with background bulk copies into shared memory; then the time of a single MMA
// instruction for a range of shapes.  Build and run on a B200:
//   nvcc -gencode arch=compute_100a,code=sm_100a -O2 -std=c++17 -o bench_mma_pattern bench_mma_pattern.cu && ./bench_mma_pattern
#include <cstdio>
#include <cuda_runtime.h>
#include "sm100_ptx.cuh"
using namespace sm100;
struct Smem { alignas(1024) uint8_t a[2][16384]; alignas(1024) uint8_t b[2][16384]; alignas(1024) uint8_t v[2][16384]; alignas(1024) uint8_t bg[2][32768];
  uint64_t bar, bars[4], bgbar[2]; uint32_t tmem_base; int abort_flag; volatile int stop; };
__global__ void __launch_bounds__(128) mix(int mode, int iters, const uint8_t* gsrc, long long* out) {
  extern __shared__ uint8_t raw[];
  Smem& s = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, warp = tid >> 5;
  for (int i = tid; i < (int)(6 * 16384) / 4; i += 128) reinterpret_cast<uint32_t*>(&s)[i] = 0;
  if (tid == 0) { s.abort_flag = 0; s.stop = 0; mbar_init(&s.bar, 1); for (int i = 0; i < 4; ++i) mbar_init(&s.bars[i], 1); mbar_init(&s.bgbar[0], 1); mbar_init(&s.bgbar[1], 1); fence_mbar_init(); }
  if (warp == 0) { tmem_alloc(&s.tmem_base, 512); tmem_relinquish(); }
  fence_proxy_async_smem(); tc_fence_before_sync(); __syncthreads(); tc_fence_after_sync();
  const uint32_t tm = s.tmem_base;
  if (tid == 0) {
    const uint32_t idesc_qk = umma_idesc_bf16(128, 128, false, false), idesc_pv = umma_idesc_bf16(128, 128, false, true);
    const uint64_t ad0 = umma_desc_sw128(smem_u32(s.a[0]), 0, 1024), bd0 = umma_desc_sw128(smem_u32(s.b[0]), 0, 1024);
    const uint64_t vd0 = umma_desc_sw128(smem_u32(s.v[0]), 16384, 1024);
    long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
      const uint32_t t = it & 1;
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        const uint64_t off = (uint64_t)((kk >> 2) * 1024 + (kk & 3) * 2);
        umma_ss(tm + t * 128, ad0 + off, bd0 + off, idesc_qk, kk > 0);
      }
      if (mode >= 1) { umma_commit(&s.bars[0]); umma_commit(&s.bars[1]); }
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) umma_ts(tm + 256 + (t ^ 1) * 128, tm + (t ^ 1) * 128 + kk * 8, vd0 + (uint64_t)(kk * 128), idesc_pv, 1);
      if (mode >= 1) { umma_commit(&s.bars[2]); umma_commit(&s.bars[3]); }
    }
    long long t1 = clock64();
    umma_commit(&s.bar);
    mbar_wait(&s.bar, 0, &s.abort_flag);
    long long t2 = clock64();
    s.stop = 1;
    if (blockIdx.x == 0) { out[0] = t1 - t0; out[1] = t2 - t0; }
  } else if (tid == 32 && mode >= 2) {
    // background bulk copies into shared memory (as the TMA producer does): 32 KB per copy, back to back
    uint32_t n = 0;
    while (!s.stop && n < 100000) {
      const int b = n & 1;
      if (n >= 2) mbar_wait(&s.bgbar[b], ((n >> 1) - 1) & 1, &s.abort_flag);
      mbar_arrive_expect_tx(&s.bgbar[b], 32768);
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(s.bg[b])), "l"(gsrc + (size_t)((n * 37 + blockIdx.x * 101) % 4096) * 32768), "r"(32768), "r"(smem_u32(&s.bgbar[b])) : "memory");
      ++n;
      if (mode == 2) { long long w = clock64(); while (clock64() - w < 1000) {} }   // ~64 KB per 2000 clk
    }
    if (n >= 1) mbar_wait(&s.bgbar[(n - 1) & 1], ((n - 1) >> 1) & 1, &s.abort_flag);
    if (n >= 2) mbar_wait(&s.bgbar[(n - 2) & 1], ((n - 2) >> 1) & 1, &s.abort_flag);
  }
  tc_fence_before_sync(); __syncthreads();
  if (warp == 0) tmem_dealloc(tm, 512);
}
// ---- time of one MMA instruction as a function of its shape: 8192 back-to-back MMAs of one shape per CTA
struct SweepSmem { alignas(1024) uint8_t a[2][16384]; alignas(1024) uint8_t b[4][16384]; uint64_t bar; uint32_t tmem_base; int abort_flag; };
template <int N, int TS, int M = 128>
__global__ void __launch_bounds__(128) shape_sweep(int iters, long long* out) {
  extern __shared__ uint8_t raw[];
  SweepSmem& s = *reinterpret_cast<SweepSmem*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, warp = tid >> 5;
  for (int i = tid; i < (int)(6 * 16384) / 4; i += 128) reinterpret_cast<uint32_t*>(&s)[i] = 0;
  if (tid == 0) { s.abort_flag = 0; mbar_init(&s.bar, 1); fence_mbar_init(); }
  if (warp == 0) { tmem_alloc(&s.tmem_base, 512); tmem_relinquish(); }
  fence_proxy_async_smem(); tc_fence_before_sync(); __syncthreads(); tc_fence_after_sync();
  const uint32_t tm = s.tmem_base;
  if (tid == 0) {
    const uint32_t idesc = umma_idesc_bf16(M, N, false, TS ? true : false);
    const uint64_t ad0 = umma_desc_sw128(smem_u32(s.a[0]), 0, 1024), bd0 = umma_desc_sw128(smem_u32(s.b[0]), TS ? 16384 : 0, 1024);
    long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        const uint64_t off = (uint64_t)((kk >> 2) * 1024 + (kk & 3) * 2);
        if (TS) umma_ts(tm + 256, tm + kk * 8, bd0 + (uint64_t)(kk * 128), idesc, 1);
        else umma_ss(tm + (it & 1) * 256, ad0 + off, bd0 + off, idesc, kk > 0);
      }
    }
    umma_commit(&s.bar);
    mbar_wait(&s.bar, 0, &s.abort_flag);
    long long t2 = clock64();
    if (blockIdx.x == 0) out[0] = t2 - t0;
  }
  tc_fence_before_sync(); __syncthreads();
  if (warp == 0) tmem_dealloc(tm, 512);
}
template <int N, int TS, int M = 128> void run_shape(long long* d) {
  size_t smem = sizeof(SweepSmem) + 1024;
  cudaFuncSetAttribute(shape_sweep<N, TS, M>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  shape_sweep<N, TS, M><<<148, 128, smem>>>(1024, d);
  cudaError_t e = cudaDeviceSynchronize();
  long long h; cudaMemcpy(&h, d, 8, cudaMemcpyDeviceToHost);
  printf("%s M=%d N=%3d K=16: %.1f clk per MMA (math floor %.0f)  %s\n", TS ? "TS" : "SS", M, N, h / 8192.0, N / 2.0, cudaGetErrorString(e));
}
int main() {
  long long* d; cudaMalloc(&d, 16);
  uint8_t* g; cudaMalloc(&g, (size_t)4096 * 32768); cudaMemset(g, 0, (size_t)4096 * 32768);
  size_t smem = sizeof(Smem) + 1024;
  cudaFuncSetAttribute(mix, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  const char* names[] = {"8 SS + 8 TS", "+ 4 commits", "+ paced background copies (64 KB / 2000 clk)", "+ unpaced background copies"};
  for (int mode = 0; mode < 4; ++mode) {
    mix<<<148, 128, smem>>>(mode, 1024, g, d);
    cudaError_t e = cudaDeviceSynchronize();
    long long h[2]; cudaMemcpy(h, d, 16, cudaMemcpyDeviceToHost);
    printf("%-46s: %.0f clk per (8 SS + 8 TS) step (ideal 1024)  %s\n", names[mode], h[1] / 1024.0, cudaGetErrorString(e));
  }
  printf("\ncycles per MMA instruction by shape (SS: both operands in shared memory, TS: A in TMEM)\n");
  run_shape<32, 0>(d); run_shape<64, 0>(d); run_shape<96, 0>(d); run_shape<128, 0>(d); run_shape<192, 0>(d); run_shape<256, 0>(d);
  run_shape<32, 1>(d); run_shape<64, 1>(d); run_shape<128, 1>(d); run_shape<256, 1>(d);
  run_shape<64, 0, 64>(d); run_shape<128, 0, 64>(d); run_shape<128, 1, 64>(d);
  return 0;
}
