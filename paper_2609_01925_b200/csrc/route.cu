// Stage 1-3a: proxy attention of the last query block, C_struct router and block scores
// (Algorithm 2; Eq. 2; Algorithm 3 lines 3-5).
//
// A_hat (128 x n per head) is never written to memory.  `proxy_partials_kernel` computes one
// 128 x 128 tile of logits per (KV head, key tile, query head of the group) with tcgen05 MMAs into
// TMEM and reduces it, one thread per proxy row, to four numbers per (row, tile): the tile-local max
// and the sums of exp(logit - max) over the entries on/below the tile diagonal, above it, and on the
// anchor keys.  Entries on/below the diagonal of key tile J belong to the diagonal band of block
// offset N_b-1-J, entries above it to offset N_b-2-J, so these sums are all the later steps need.
// Every row thread also carries the running maximum and sum of its row over the tiles its CTA visits; the
// last CTA of a KV group to finish merges these per-CTA statistics into the global row maximum and
// 1 / row sum.  One more kernel (`tile_sums_kernel`) turns the partials into per-tile masses across rows
// with warp-shuffle reductions, and the last of its CTAs to finish a head adds up p_s and C_struct and
// sets the routing label.  All reductions run in a fixed order.
#include <cstdio>
#include <mutex>

#include <algorithm>
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace crisp {
using namespace sm100;

namespace {

constexpr int kChunk = 16;  // key tiles per CTA in the merge kernels

// ---- packed fp32x2 arithmetic (two values per instruction on the FMA pipe)
__device__ __forceinline__ uint64_t pack2f(float lo, float hi) {
  uint64_t v;
  asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
  return v;
}
__device__ __forceinline__ void unpack2f(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2f(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2f(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

struct RoutePtrs {
  float* pm;       // [hq][nb][128] tile-local max of the scaled logits (base-2 units)
  float* plo;      // [hq][nb][128] sum of 2^(x - max) over entries with key offset <= row
  float* pup;      // [hq][nb][128] ... over entries with key offset > row
  float* phi;      // [hq][nb][128] third band, only when n is not a multiple of 128 (see proxy_partials_kernel)
  float* panc;     // [hq][slots][128] ... over anchor keys of the tile
  float* cm;       // [hq][n_slices][128] row maximum over the tiles one proxy CTA visited
  float* cl;       // [hq][n_slices][128] row sum relative to that maximum
  float* row_m;    // [hq][128] global row max
  float* row_invl; // [hq][128] 1 / global row sum
  float* slo;      // [hq][nb] mass (over rows) on/below the tile diagonal
  float* sup;      // [hq][nb] mass above the tile diagonal
  float* shi;      // [hq][nb] mass of the third band (ragged n only)
  int* group_done; // [proxy grid.y] CTAs of a (KV head, head chunk) group that finished (zeroed per call)
  int* head_done;  // [hq] CTAs of tile_sums that finished a head (zeroed per call)
  size_t zero_bytes;  // header + counters
  int n_chunks;    // chunks of kChunk key tiles (tile_sums)
  int n_slices;    // proxy CTAs per group = entries of cm / cl per (head, row)
};

constexpr int kProxyHeads = 4;  // query heads of one KV group handled by one CTA (their proxy queries stay in shared memory)

struct ProxySmem {
  alignas(1024) uint8_t q[kProxyHeads][2][16384];  // [head][half] proxy queries, resident for the CTA's lifetime
  alignas(1024) uint8_t k[2][2][16384];            // [buffer][half] key tiles, two 64-column halves, 128-byte swizzle
  uint64_t bar_q;
  uint64_t bar_k_full[2], bar_k_free[2];
  uint64_t bar_s_full[4], bar_s_free[4];
  uint32_t tmem_base;
  int abort_flag;
  int is_last;
};

// Persistent CTAs, one per SM.  A CTA owns up to four query heads of one KV group - their 128 proxy queries
// are loaded once and stay in shared memory - and walks over every S-th key tile, S being the number of CTAs of
// its group (the groups share the SMs evenly; SMs left over go to the first groups): TMA brings the K
// tile in (two buffers, the load of the tile after next is issued while the current one is worked on), one
// thread issues a 128 x 128 x 128 tcgen05 MMA per head into that head's TMEM buffer, and four groups of four
// warps (one group per head, one thread per proxy row) reduce the logits to the tile partials.  The row threads
// wait on the latencies of their own chain (TMEM load, row maximum, dependent exp2 / add pairs), not on MUFU
// throughput, so what counts is the number of warps per scheduler: a thread reads its row in two halves of 64
// keys - half a row of registers - which lets four warps per scheduler fit (the maximum needs a first pass over
// both halves; the second half stays in registers for the sums, the first is read again).
// kRagged: n is not a multiple of 128 (third band possible); the aligned instantiation drops its predicates.
constexpr int kProxyThreads = 32 * (4 * kProxyHeads + 1);

template <bool kRagged>
__global__ void __launch_bounds__(kProxyThreads, 1)
proxy_partials_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                      const Dims d, const RoutePtrs w, int* status, int n_head_chunks, int base_slices,
                      int extra_groups) {
  pdl_enter();
  extern __shared__ uint8_t smem_raw[];
  ProxySmem& s = *reinterpret_cast<ProxySmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = d.group;
  // CTA -> (group, slice): the first extra_groups groups have base_slices + 1 CTAs, the others base_slices
  int grp, sl, stride;
  {
    const int b = blockIdx.x, big = extra_groups * (base_slices + 1);
    if (b < big) {
      grp = b / (base_slices + 1);
      sl = b % (base_slices + 1);
      stride = base_slices + 1;
    } else {
      grp = extra_groups + (b - big) / base_slices;
      sl = (b - big) % base_slices;
      stride = base_slices;
    }
  }
  const int kvh = grp / n_head_chunks, g0 = (grp % n_head_chunks) * kProxyHeads;
  const int gc = min(kProxyHeads, G - g0);            // heads of this CTA
  const int n_my_tiles = sl < d.nb ? (d.nb - 1 - sl) / stride + 1 : 0;
  constexpr int kIssuerWarp = 4 * kProxyHeads;

  if (tid == 0) {
    s.abort_flag = 0;
    mbar_init(&s.bar_q, 1);
    for (int b = 0; b < 2; ++b) {
      mbar_init(&s.bar_k_full[b], 1);
      mbar_init(&s.bar_k_free[b], 1);
    }
    for (int b = 0; b < 4; ++b) {
      mbar_init(&s.bar_s_full[b], 1);
      mbar_init(&s.bar_s_free[b], 4);  // one arrival per warp of the group that reads the buffer
    }
    fence_mbar_init();
  }
  if (warp == kIssuerWarp) {
    tmem_alloc(&s.tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tm = s.tmem_base;

  if (warp == kIssuerWarp) {
    if (lane == 0 && n_my_tiles > 0) {
      // ---- producer + MMA issuer
      prefetch_tmap(&tmap_q);
      prefetch_tmap(&tmap_k);
      auto load_k = [&](int n) {
        const int J = sl + n * stride, kb = n & 1;
        mbar_arrive_expect_tx(&s.bar_k_full[kb], 32768);
        tma_load_3d(s.k[kb][0], &tmap_k, &s.bar_k_full[kb], 0, kvh, J * kBlock);
        tma_load_3d(s.k[kb][1], &tmap_k, &s.bar_k_full[kb], 64, kvh, J * kBlock);
      };
      load_k(0);
      mbar_arrive_expect_tx(&s.bar_q, 32768u * gc);
      for (int g = 0; g < gc; ++g) {
        tma_load_3d(s.q[g][0], &tmap_q, &s.bar_q, 0, kvh * G + g0 + g, d.n - kBlock);
        tma_load_3d(s.q[g][1], &tmap_q, &s.bar_q, 64, kvh * G + g0 + g, d.n - kBlock);
      }
      if (n_my_tiles > 1) load_k(1);
      bool ok = mbar_wait(&s.bar_q, 0, &s.abort_flag);
      constexpr uint32_t idesc = umma_idesc_bf16(128, 128, false, false);
      const uint64_t q_desc0 = umma_desc_sw128(smem_u32(s.q[0][0]), 0, 1024);
      const uint64_t k_desc0 = umma_desc_sw128(smem_u32(s.k[0][0]), 0, 1024);
      for (int n = 0; n < n_my_tiles && ok; ++n) {
        const int kb = n & 1;
        ok = mbar_wait(&s.bar_k_full[kb], (n >> 1) & 1, &s.abort_flag);
        for (int g = 0; g < gc && ok; ++g) {
          // head g's logits go to TMEM buffer g, which its group has finished reading for the previous tile
          if (n > 0) ok = mbar_wait(&s.bar_s_free[g], (n - 1) & 1, &s.abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          // descriptors: only the 14-bit start-address field moves (head: +32 KB, buffer: +32 KB, K step kk:
          // 16 KB per 64-dim half, 32 B per step inside the swizzle atom), so an MMA costs two integer adds
          const uint64_t ad0 = q_desc0 + static_cast<uint64_t>(g) * 2048u, bd0 = k_desc0 + static_cast<uint64_t>(kb) * 2048u;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            constexpr uint32_t kHalf = 16384 >> 4, kStep = 32 >> 4;
            const uint64_t off = static_cast<uint64_t>((kk >> 2) * kHalf + (kk & 3) * kStep);
            umma_ss(tm + g * 128, ad0 + off, bd0 + off, idesc, kk > 0);
          }
          umma_commit(&s.bar_s_full[g]);
          // As early in this tile as the pipe allows, refill the other buffer (the previous tile's, whose MMAs
          // were issued a whole tile ago) with the next tile, so its latency hides behind this tile's work.
          if (g == 0 && n >= 1 && n + 1 < n_my_tiles) {
            ok = mbar_wait(&s.bar_k_free[kb ^ 1], ((n - 1) >> 1) & 1, &s.abort_flag);
            if (ok) load_k(n + 1);
          }
        }
        if (!ok) break;
        umma_commit(&s.bar_k_free[kb]);  // the K buffer is free once this tile's MMAs have read it
      }
    }
    __syncwarp();
  } else if ((warp >> 2) < gc) {
    // ---- one thread per proxy row; group gr = warps 4 gr .. 4 gr + 3 takes head gr of the CTA
    const int gr = warp >> 2;
    const int i = tid & 127;
    const int wq = warp & 3;  // warp within the group = TMEM sub-partition = rows 32 wq .. 32 wq + 31
    // Offset of proxy row i to local key jl of a tile: o = t_i - j = q * 128 + (rho + i - jl) with
    // q = nfull - 1 - J and rho = n mod 128.  The entry is visible iff o >= 0 and belongs to the diagonal
    // band of block offset floor(o / 128), which is q - 1 ("up": jl > i + rho), q ("lo") or q + 1
    // ("hi": jl <= i + rho - 128, possible only when rho > 0).  A band with a negative offset is invisible.
    const int a_thr = i + d.rho;           // jl <= a_thr  <=>  not in the "up" band
    const int b_thr = i + d.rho - kBlock;  // jl <= b_thr  <=>  in the "hi" band
    const uint32_t s_addr = tm + (static_cast<uint32_t>(wq * 32) << 16) + gr * 128;
    const int h = kvh * G + g0 + gr;
    bool ok = true;
    // running maximum and sum of this row over the CTA's tiles
    float run_m = -INFINITY, run_l = 0.f;
    for (int n = 0; n < n_my_tiles && ok; ++n) {
      const int J = sl + n * stride;
      const int qoff = d.nfull - 1 - J;
      const bool vis_up = qoff - 1 >= 0, vis_lo = qoff >= 0;  // "hi" (q + 1 >= 0) is visible whenever it is non-empty
      const int js = min(max(d.w_sink - J * kBlock, 0), kBlock);         // anchor: local key < js
      const int jl = min(max(d.n - d.w_local - J * kBlock, 0), kBlock);  // anchor: local key >= jl
      const bool has_slot = (J < d.n_sink_tiles) || (J >= d.first_local_tile);
      const int slot = (J < d.n_sink_tiles) ? J : d.n_sink_tiles + (J - d.first_local_tile);
      if (!mbar_wait(&s.bar_s_full[gr], n & 1, &s.abort_flag)) {
        ok = false;
        break;
      }
      tc_fence_after_sync();
      const bool interior = !kRagged && vis_up;  // every key visible, band of key jl decided by jl <= i alone
      uint32_t r[2][32];
      // ---- first pass: the row maximum over the visible keys, half A (keys 0-63) then half B (64-127)
      float mx = -INFINITY;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        tmem_ld_x32(s_addr + half * 64, r[0]);
        tmem_ld_x32(s_addr + half * 64 + 32, r[1]);
        tmem_ld_wait();
        if (interior) {
          float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
          for (int c = 0; c < 2; ++c)
#pragma unroll
            for (int t = 0; t < 32; t += 2) {
              m0 = fmaxf(m0, __uint_as_float(r[c][t]));
              m1 = fmaxf(m1, __uint_as_float(r[c][t + 1]));
            }
          mx = fmaxf(mx, fmaxf(m0, m1));
        } else {
#pragma unroll
          for (int c = 0; c < 2; ++c)
#pragma unroll
            for (int t = 0; t < 32; ++t) {
              const int j = half * 64 + c * 32 + t;
              const bool visible = (kRagged && j <= b_thr) || (j <= a_thr ? vis_lo : vis_up);
              if (visible) mx = fmaxf(mx, __uint_as_float(r[c][t]));
            }
        }
      }
      mx *= d.scale_log2;  // (the scale is positive)
      // a row may see no key of this tile (ragged n: the tiles around the proxy block): leave a neutral partial
      const bool any = mx > -INFINITY;
      if (!any) mx = -1e30f;
      float lo = 0.f, up = 0.f, hi = 0.f, anc = 0.f;
      // ---- second pass: the sums, half B from the registers it is still in, then half A read again
#pragma unroll
      for (int pass = 0; pass < 2; ++pass) {
        const int half = 1 - pass;
        if (pass == 1) {
          tmem_ld_x32(s_addr, r[0]);
          tmem_ld_x32(s_addr + 32, r[1]);
          tmem_ld_wait();
          // the buffer has been read for good: the next tile's logits of this head may come in
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&s.bar_s_free[gr]);
        }
        if (interior) {
          // Rows of warp wq lie in [32 wq, 32 wq + 31], so a 32-key chunk c lies wholly on/below the diagonal
          // for c < wq and wholly above it for c > wq: only the chunk c == wq needs a per-key test.
          const uint64_t scale2 = pack2f(d.scale_log2, d.scale_log2), negm2 = pack2f(-mx, -mx);
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            const int c = 2 * half + cc;
            if (c != wq) {
              // the whole chunk lies in one band: packed fp32x2 arithmetic, no per-key test
              uint64_t sa = pack2f(0.f, 0.f), sb = pack2f(0.f, 0.f);
#pragma unroll
              for (int t = 0; t < 32; t += 4) {
                float a0, a1, b0, b1;
                unpack2f(fma2f(pack2f(__uint_as_float(r[cc][t]), __uint_as_float(r[cc][t + 1])), scale2, negm2), a0, a1);
                unpack2f(fma2f(pack2f(__uint_as_float(r[cc][t + 2]), __uint_as_float(r[cc][t + 3])), scale2, negm2), b0, b1);
                sa = add2f(sa, pack2f(ex2(a0), ex2(a1)));
                sb = add2f(sb, pack2f(ex2(b0), ex2(b1)));
              }
              float x0, x1, y0, y1;
              unpack2f(sa, x0, x1);
              unpack2f(sb, y0, y1);
              const float sum = (x0 + x1) + (y0 + y1);
              if (c < wq) {
                lo += sum;
              } else {
                up += sum;
              }
            } else {
              // the chunk the diagonal crosses: key 32 c + t is on/below it iff t <= i - 32 c
              const int il = i - 32 * c;
              float d0 = 0.f, d1 = 0.f, u0 = 0.f, u1 = 0.f;
#pragma unroll
              for (int t = 0; t < 32; t += 2) {
                const float e0 = ex2(fmaf(__uint_as_float(r[cc][t]), d.scale_log2, -mx));
                const float e1 = ex2(fmaf(__uint_as_float(r[cc][t + 1]), d.scale_log2, -mx));
                d0 += t <= il ? e0 : 0.f;
                u0 += t <= il ? 0.f : e0;
                d1 += t + 1 <= il ? e1 : 0.f;
                u1 += t + 1 <= il ? 0.f : e1;
              }
              lo += d0 + d1;
              up += u0 + u1;
            }
          }
          if (has_slot) {
            // the few tiles that hold anchor keys (sinks, the local window) take another pass for their sum
#pragma unroll
            for (int cc = 0; cc < 2; ++cc)
#pragma unroll
              for (int t = 0; t < 32; ++t) {
                const int j = half * 64 + cc * 32 + t;
                if (j < js || j >= jl) anc += ex2(fmaf(__uint_as_float(r[cc][t]), d.scale_log2, -mx));
              }
          }
        } else {
#pragma unroll
          for (int cc = 0; cc < 2; ++cc)
#pragma unroll
            for (int t = 0; t < 32; ++t) {
              const int j = half * 64 + cc * 32 + t;
              const float e = ex2(fmaf(__uint_as_float(r[cc][t]), d.scale_log2, -mx));
              const bool in_hi = kRagged && j <= b_thr, in_lo = !in_hi && j <= a_thr, in_up = j > a_thr;
              const bool visible = in_hi || (in_lo && vis_lo) || (in_up && vis_up);
              hi += in_hi ? e : 0.f;
              lo += (in_lo && vis_lo) ? e : 0.f;
              up += (in_up && vis_up) ? e : 0.f;
              anc += (visible && (j < js || j >= jl)) ? e : 0.f;
            }
        }
      }
      if (!any) lo = up = hi = anc = 0.f;
      {
        const float sum = lo + up + hi;
        const float nm = fmaxf(run_m, mx);
        run_l = run_l * ex2(run_m - nm) + sum * ex2(mx - nm);
        run_m = nm;
      }
      const size_t off = (static_cast<size_t>(h) * d.nb + J) * kBlock + i;
      w.pm[off] = mx;
      w.plo[off] = lo;
      w.pup[off] = up;
      if (kRagged) w.phi[off] = hi;
      if (has_slot) w.panc[(static_cast<size_t>(h) * d.n_anchor_slots + slot) * kBlock + i] = anc;
    }
    // this CTA's share of the row statistics
    {
      const size_t o = (static_cast<size_t>(h) * w.n_slices + sl) * kBlock + i;
      w.cm[o] = run_m;
      w.cl[o] = run_l;
    }
  }
  tc_fence_before_sync();
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    if (s.abort_flag) atomicExch(status, CRISP_ERR_DEVICE_TIMEOUT);
    s.is_last = atomicAdd(&w.group_done[grp], 1) == stride - 1;
  }
  if (warp == kIssuerWarp) tmem_dealloc(tm, 512);
  __syncthreads();
  if (!s.is_last) return;
  // The last CTA of the group to finish merges the per-CTA statistics (written by other CTAs: read from L2)
  // into the global row maximum and 1 / row sum of the group's heads.
  __threadfence();
  for (int item = tid; item < gc * kBlock; item += blockDim.x) {
    const int h = kvh * G + g0 + item / kBlock, i = item % kBlock;
    float M = -INFINITY, L = 0.f;
    for (int c = 0; c < stride; ++c) {
      const size_t o = (static_cast<size_t>(h) * w.n_slices + c) * kBlock + i;
      const float m = __ldcg(w.cm + o), l = __ldcg(w.cl + o);
      const float nm = fmaxf(M, m);
      L = L * ex2(M - nm) + l * ex2(m - nm);
      M = nm;
    }
    w.row_m[h * kBlock + i] = M;
    w.row_invl[h * kBlock + i] = 1.0f / L;
  }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Per (head, chunk): one warp per key tile sums the normalised masses over the 128 proxy rows.  The last CTA of
// a head to finish then forms the slash scores from the two (three) triangle sums, C_struct from the anchor
// partials, and the routing label.
__global__ void __launch_bounds__(128) tile_sums_kernel(const Dims d, const RoutePtrs w, float* __restrict__ p_v,
                                                        float* __restrict__ p_s, float* __restrict__ c_struct,
                                                        int32_t* __restrict__ pattern) {
  pdl_enter();
  const int h = blockIdx.y, chunk = blockIdx.x;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  float M[4], invl[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    M[r] = w.row_m[h * kBlock + lane + 32 * r];
    invl[r] = w.row_invl[h * kBlock + lane + 32 * r] * (1.0f / kBlock);
  }
  const int j0 = chunk * kChunk, j1 = min(j0 + kChunk, d.nb);
  for (int J = j0 + warp; J < j1; J += 4) {
    const size_t base = (static_cast<size_t>(h) * d.nb + J) * kBlock + lane;
    float lo = 0.f, up = 0.f, hi = 0.f;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const float wgt = ex2(w.pm[base + 32 * r] - M[r]) * invl[r];
      lo += wgt * w.plo[base + 32 * r];
      up += wgt * w.pup[base + 32 * r];
      if (d.rho > 0) hi += wgt * w.phi[base + 32 * r];
    }
    lo = warp_sum(lo);
    up = warp_sum(up);
    hi = warp_sum(hi);
    if (lane == 0) {
      w.slo[static_cast<size_t>(h) * d.nb + J] = lo;
      w.sup[static_cast<size_t>(h) * d.nb + J] = up;
      w.shi[static_cast<size_t>(h) * d.nb + J] = hi;
      p_v[static_cast<size_t>(h) * d.nb + J] = (lo + up) + hi;
    }
  }
  __shared__ int is_last;
  __shared__ float red[4];
  __threadfence();
  __syncthreads();
  if (tid == 0) is_last = atomicAdd(&w.head_done[h], 1) == static_cast<int>(gridDim.x) - 1;
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  // ---- the head's last CTA.  The tile sums came from other CTAs: read them from L2.
  const float* slo = w.slo + static_cast<size_t>(h) * d.nb;
  const float* sup = w.sup + static_cast<size_t>(h) * d.nb;
  const float* shi = w.shi + static_cast<size_t>(h) * d.nb;
  // band of block offset s: "lo" of tile nfull-1-s, "up" of tile nfull-2-s, "hi" of tile nfull-s
  for (int sidx = tid; sidx < d.nb; sidx += blockDim.x) {
    const int jlo = d.nfull - 1 - sidx, jup = d.nfull - 2 - sidx, jhi = d.nfull - sidx;
    float v = 0.f;
    if (jlo >= 0 && jlo < d.nb) v += __ldcg(slo + jlo);
    if (jup >= 0 && jup < d.nb) v += __ldcg(sup + jup);
    if (d.rho > 0 && jhi >= 0 && jhi < d.nb) v += __ldcg(shi + jhi);
    p_s[static_cast<size_t>(h) * d.nb + sidx] = v;
  }
  float acc = 0.f;
  {
    const float Mr = w.row_m[h * kBlock + tid];
    const float inv = w.row_invl[h * kBlock + tid] * (1.0f / kBlock);
    for (int slot = 0; slot < d.n_anchor_slots; ++slot) {
      const int J = slot < d.n_sink_tiles ? slot : d.first_local_tile + (slot - d.n_sink_tiles);
      const float m = w.pm[(static_cast<size_t>(h) * d.nb + J) * kBlock + tid];
      acc += ex2(m - Mr) * inv * w.panc[(static_cast<size_t>(h) * d.n_anchor_slots + slot) * kBlock + tid];
    }
    acc = warp_sum(acc);
    if (lane == 0) red[warp] = acc;
  }
  __syncthreads();
  if (tid == 0) {
    const float c = (red[0] + red[1]) + (red[2] + red[3]);
    c_struct[h] = c;
    int pat = (c >= d.tau) ? CRISP_PATTERN_VS : CRISP_PATTERN_PE;
    if (d.force_pattern == 1) pat = CRISP_PATTERN_VS;
    if (d.force_pattern == 2) pat = CRISP_PATTERN_PE;
    pattern[h] = pat;
  }
}

// How the proxy kernel's grid is laid out: one CTA per SM; the (KV head, chunk of four query heads) groups share
// the SMs evenly, each group's CTAs split its key tiles.
struct ProxyGrid {
  int n_head_chunks, groups, slices, extra;  // `extra` groups have slices + 1 CTAs
};
ProxyGrid proxy_grid(const Dims& d, int n_sm) {
  ProxyGrid g;
  g.n_head_chunks = (d.group + kProxyHeads - 1) / kProxyHeads;
  g.groups = d.hkv * g.n_head_chunks;
  g.slices = n_sm / g.groups;
  g.extra = n_sm % g.groups;  // the SMs the even split leaves over go to the first groups
  if (g.slices < 1) {
    g.slices = 1;
    g.extra = 0;
  }
  if (g.slices >= d.nb) {
    g.slices = d.nb;
    g.extra = 0;
  }
  return g;
}
// The workspace is sized without knowing the device: room for the CTAs of a 160-SM part; a larger device simply
// runs with that many CTAs per group.
constexpr int kSizedForSms = 160;

RoutePtrs carve(const Dims& d, void* ws) {
  RoutePtrs w;
  uint8_t* p = static_cast<uint8_t*>(ws) + kWsHeader;
  auto take = [&](size_t n_floats) {
    float* r = reinterpret_cast<float*>(p);
    p += align_up(n_floats * sizeof(float), 256);
    return r;
  };
  // counters first: one memset clears them together with the header
  const int n_head_chunks = (d.group + kProxyHeads - 1) / kProxyHeads;
  w.group_done = reinterpret_cast<int*>(take(static_cast<size_t>(d.hkv) * n_head_chunks));
  w.head_done = reinterpret_cast<int*>(take(d.hq));
  w.zero_bytes = static_cast<size_t>(p - static_cast<uint8_t*>(ws));
  w.n_chunks = (d.nb + kChunk - 1) / kChunk;
  w.n_slices = max(1, min(kSizedForSms / (d.hkv * n_head_chunks), d.nb));
  const size_t part = static_cast<size_t>(d.hq) * d.nb * kBlock;
  w.pm = take(part);
  w.plo = take(part);
  w.pup = take(part);
  w.phi = d.rho > 0 ? take(part) : nullptr;  // third band: only for lengths that are not multiples of 128
  w.panc = take(static_cast<size_t>(d.hq) * d.n_anchor_slots * kBlock);
  w.cm = take(static_cast<size_t>(d.hq) * w.n_slices * kBlock);
  w.cl = take(static_cast<size_t>(d.hq) * w.n_slices * kBlock);
  w.row_m = take(static_cast<size_t>(d.hq) * kBlock);
  w.row_invl = take(static_cast<size_t>(d.hq) * kBlock);
  w.slo = take(static_cast<size_t>(d.hq) * d.nb);
  w.sup = take(static_cast<size_t>(d.hq) * d.nb);
  w.shi = take(static_cast<size_t>(d.hq) * d.nb);
  return w;
}

}  // namespace

size_t route_ws_bytes(const Dims& d) {
  RoutePtrs w = carve(d, nullptr);
  return reinterpret_cast<size_t>(w.shi) + align_up(static_cast<size_t>(d.hq) * d.nb * sizeof(float), 256);
}

int launch_route(const Dims& d, const void* q, const void* k, void* ws, float* c_struct, int32_t* pattern,
                 float* p_v, float* p_s, cudaStream_t stream) {
  RoutePtrs w = carve(d, ws);
  int* status = static_cast<int*>(ws);
  CRISP_CUDA_TRY(cudaMemsetAsync(ws, 0, w.zero_bytes, stream), "route: clear status and counters");
  CUtensorMap tq, tk;
  int rc = make_tmap_bf16_nhd(&tq, q, d.n, d.hq);
  if (rc != CRISP_OK) return rc;
  rc = make_tmap_bf16_nhd(&tk, k, d.n, d.hkv);
  if (rc != CRISP_OK) return rc;
  const size_t smem = sizeof(ProxySmem) + 1024;
  auto* proxy = d.rho > 0 ? proxy_partials_kernel<true> : proxy_partials_kernel<false>;
  CRISP_CUDA_TRY(cudaFuncSetAttribute(proxy, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)),
                 "route: smem attribute");
  int dev = 0, n_sm = 0;
  CRISP_CUDA_TRY(cudaGetDevice(&dev), "route: current device");
  CRISP_CUDA_TRY(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev), "route: SM count");
  ProxyGrid g = proxy_grid(d, n_sm);
  if (g.slices + (g.extra > 0 ? 1 : 0) > w.n_slices) {
    g.slices = std::min(g.slices, w.n_slices);
    g.extra = 0;
  }
  CRISP_KERNEL("proxy", stream,
               launch_pdl(proxy, dim3(g.slices * g.groups + g.extra), dim3(kProxyThreads), smem, stream, tq, tk, d, w,
                          status, g.n_head_chunks, g.slices, g.extra));
  CRISP_KERNEL("tile_sums", stream, launch_pdl(tile_sums_kernel, dim3(w.n_chunks, d.hq), dim3(128), 0, stream, d, w, p_v, p_s, c_struct, pattern));
  CRISP_CUDA_TRY(cudaGetLastError(), "route: launch");
  return CRISP_OK;
}

// ------------------------------------------------------------------------------------------------
// Routing for callers that cannot allocate device memory.  Same kernels as launch_route; the scratch
// lives in a fixed array that is part of the loaded library image on every GPU.
// ------------------------------------------------------------------------------------------------
namespace {
constexpr size_t kStaticScratchBytes = CRISP_ROUTE_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_route_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_addr[kMaxDevices] = {};  // device address of g_route_scratch, per device ordinal
}  // namespace

int launch_route_static(const Dims& d, const void* q, const void* k, float* c_struct, int32_t* pattern,
                        float* p_v, float* p_s, int32_t* device_status, cudaStream_t stream) {
  const size_t need = route_ws_bytes(d);
  if (need > kStaticScratchBytes) {
    char msg[160];
    std::snprintf(msg, sizeof(msg),
                  "crisp_route_static: this problem needs %zu bytes of scratch, the built-in array holds %zu",
                  need, kStaticScratchBytes);
    set_cu_error(msg);
    return CRISP_ERR_UNSUPPORTED;
  }
  int dev = 0;
  CRISP_CUDA_TRY(cudaGetDevice(&dev), "route_static: current device");
  if (dev < 0 || dev >= kMaxDevices) {
    set_cu_error("crisp_route_static: device ordinal out of range");
    return CRISP_ERR_UNSUPPORTED;
  }
  void* scratch = nullptr;
  {
    // In host code the array's name is only a handle; the kernels need its address on THIS device.
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (g_scratch_addr[dev] == nullptr) {
      void* p = nullptr;
      CRISP_CUDA_TRY(cudaGetSymbolAddress(&p, g_route_scratch), "route_static: symbol address");
      g_scratch_addr[dev] = p;
    }
    scratch = g_scratch_addr[dev];
  }
  // launch_route clears the status word at the start of the scratch; every other byte it reads is
  // written earlier in the same call, so stale contents of the previous call are never observed.
  const int rc = launch_route(d, q, k, scratch, c_struct, pattern, p_v, p_s, stream);
  if (rc != CRISP_OK) return rc;
  if (device_status)
    CRISP_CUDA_TRY(cudaMemcpyAsync(device_status, scratch, sizeof(int32_t), cudaMemcpyDeviceToDevice, stream),
                   "route_static: status copy");
  return CRISP_OK;
}

}  // namespace crisp
