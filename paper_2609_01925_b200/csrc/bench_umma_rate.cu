// Stand-alone micro-benchmark: cycles per tcgen05.mma (bf16, M = 128) for shared-memory and TMEM A
// operands and N = 128 / 256, one CTA per SM.  Build and run on a B200:
//   nvcc -gencode arch=compute_100a,code=sm_100a -O2 -std=c++17 -o bench_umma_rate bench_umma_rate.cu && ./bench_umma_rate
#include <cstdio>
#include <cstdlib>
#include <vector>
#include <cuda_runtime.h>
#include "sm100_ptx.cuh"
using namespace sm100;

struct Smem {
  alignas(1024) uint8_t a[2][16384];
  alignas(1024) uint8_t b[4][16384];
  uint64_t bar;
  uint32_t tmem_base;
  int abort_flag;
};

// mode 0: SS M128 N128 K-major B; 1: SS N256; 2: TS N128 with MN-major B (like P*V); 3: TS N256; 4: SS N128 MN-major B
__global__ void __launch_bounds__(128) rate(int mode, int iters, long long* out) {
  extern __shared__ uint8_t raw[];
  Smem& s = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, warp = tid >> 5;
  for (int i = tid; i < (int)sizeof(Smem) / 4 - 64; i += 128) reinterpret_cast<uint32_t*>(&s)[i] = 0;
  if (tid == 0) { s.abort_flag = 0; mbar_init(&s.bar, 1); fence_mbar_init(); }
  if (warp == 0) { tmem_alloc(&s.tmem_base, 512); tmem_relinquish(); }
  fence_proxy_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tm = s.tmem_base;
  if (tid == 0) {
    const int N = (mode == 1 || mode == 3) ? 256 : 128;
    const bool bmn = (mode == 2 || mode == 3 || mode == 4);
    const uint32_t idesc = umma_idesc_bf16(128, N, false, bmn);
    const uint64_t ad0 = umma_desc_sw128(smem_u32(s.a[0]), 0, 1024);
    const uint64_t bd0 = bmn ? umma_desc_sw128(smem_u32(s.b[0]), 16384, 1024) : umma_desc_sw128(smem_u32(s.b[0]), 0, 1024);
    long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        if (mode == 2 || mode == 3) {
          umma_ts(tm + 256, tm + kk * 8, bd0 + (uint64_t)(kk * 128), idesc, 1);
        } else if (mode == 4) {
          umma_ss(tm + 256, ad0 + (uint64_t)((kk >> 2) * 1024 + (kk & 3) * 2), bd0 + (uint64_t)(kk * 128), idesc, 1);
        } else {
          const uint64_t off = (uint64_t)((kk >> 2) * 1024 + (kk & 3) * 2);
          umma_ss(tm + 0, ad0 + off, bd0 + off, idesc, 1);
        }
      }
    }
    long long t1 = clock64();
    umma_commit(&s.bar);
    mbar_wait(&s.bar, 0, &s.abort_flag);
    long long t2 = clock64();
    if (blockIdx.x == 0) { out[0] = t1 - t0; out[1] = t2 - t0; }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tm, 512);
}

int main() {
  long long* d; cudaMalloc(&d, 16);
  size_t smem = sizeof(Smem) + 1024;
  cudaFuncSetAttribute(rate, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  const char* names[] = {"SS M128 N128 (K-major B)", "SS M128 N256", "TS M128 N128 (MN-major B)", "TS M128 N256", "SS M128 N128 MN-major B"};
  for (int mode = 0; mode < 5; ++mode) {
    for (int grid : {1, 148}) {
      int iters = 512;
      rate<<<grid, 128, smem>>>(mode, iters, d);
      cudaError_t e = cudaDeviceSynchronize();
      long long h[2]; cudaMemcpy(h, d, 16, cudaMemcpyDeviceToHost);
      int N = (mode == 1 || mode == 3) ? 256 : 128;
      double per = (double)h[1] / (iters * 8);
      printf("%-28s grid %3d: issue %.1f clk/MMA, complete %.1f clk/MMA  (ideal %d)  %s\n", names[mode], grid, (double)h[0] / (iters * 8), per, N / 2, cudaGetErrorString(e));
    }
  }
  return 0;
}
