// Stage 3b-3c: block selection and expansion into per-query-block key-block lists.
//
//   VS heads  (Algorithm 3 lines 6-12 / Eq. 3-4; Algorithm 6 when selector == 1; the median floor of
//     Appendix H when selector == 2):
//     `select_vs_kernel`, one CTA per (head, direction), keeps p_d in shared memory, computes the
//     noise floor, the budget k_d and the top-k_d set (ties to the lower index) as a bitmap.
//   PE heads  (Algorithm 4): block means of Q and K (`pool_kernel`), pooled logits (`pe_logits_kernel`),
//     causal row softmax normalised by the total (`pe_normalise_kernel`), then the gamma cut WITHOUT a
//     sort: a three-level radix histogram over the fp32 bit patterns (`pe_hist_kernel`,
//     `pe_cut_kernel`), with masses in exact fixed point, finds the value at the cut and how many
//     entries tied with it are taken (ties in row-major order).
//   Expansion + compaction: per (head, query block) a bitmap over key blocks is formed from the
//     vertical bitmap, the shifted slash bitmap and the forced blocks {0, m}; popcounts give the row
//     lengths (`count_vs_kernel`), one scan gives row_ptr (`scan_rows_kernel`), a second pass writes the
//     ascending column lists (`fill_kernel`).  No atomics touch the lists, so they are reproducible.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace crisp {
using namespace sm100;

namespace {

constexpr int kL0Bins = 2048, kL1Bins = 2048, kL2Bins = 512;  // key bits 30..20, 19..9, 8..0
constexpr int kHistStride = kL0Bins + kL1Bins + kL2Bins;

// Masses are accumulated in 2^-60 fixed point: integer adds are exact and order independent, so the
// histograms (built with atomics) and everything derived from them are reproducible.
constexpr float kMassScale = 1152921504606846976.0f;  // 2^60

struct CutState {                 // per head, device memory
  unsigned int prefix;            // key bits fixed so far
  unsigned int cutkey;            // final: fp32 bit pattern of the value at the cut
  unsigned long long mass_above;  // mass (fixed point) of entries strictly above the current prefix range
  long long take;                 // number of entries equal to cutkey that are selected; -1 = everything
};

struct SelectPtrs {
  uint32_t* selv;   // [hq][words] vertical bitmap
  uint32_t* selsr;  // [hq][words + 2] reversed slash bitmap: bit x = S_s contains N_b-1-x
  float* kbar;      // [hkv][nb][128]
  float* qbar;      // [hq][nb][128]
  __nv_bfloat16* ksplit;  // [3][nb][hkv][128] block means of K as three bf16 terms (hi + mid + lo = the fp32 mean)
  __nv_bfloat16* qsplit;  // [3][nb][hq][128]  the same for Q
  float* amat;      // [hq][nb][nb] pooled map (row m uses columns 0..m)
  unsigned int* hcount;  // [hq][kHistStride]
  unsigned long long* hmass;  // [hq][kHistStride] fixed-point mass per bin
  CutState* cut;         // [hq]
  int* n_gt;        // [hq][nb]
  int* n_eq;        // [hq][nb]
  int* flags;       // [hq][nb] bit0: a[m][0] > cut, bit1: == cut, bit2: a[m][m] > cut, bit3: == cut
  int* take;        // [hq][nb] ties of row m that are selected
  int* counts;      // [hq][nb] row lengths
  int words;
};

__device__ __forceinline__ int warp_sum_i(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Block-wide sum in a fixed order (warp shuffles, then the warp totals in warp order).
template <typename T>
__device__ T block_sum(T v, T* scratch /* >= 32 */) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  T total = 0;
  for (int wdx = 0; wdx < nw; ++wdx) total += scratch[wdx];
  return total;
}

// ------------------------------------------------------------------------------------------------
// VS heads: budget and top-k per direction
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
select_vs_kernel(const Dims d, const int32_t* __restrict__ pattern, const float* __restrict__ p_v,
                 const float* __restrict__ p_s, const SelectPtrs w) {
  extern __shared__ uint8_t sm_raw[];
  const int nb = d.nb;
  double* sorted = reinterpret_cast<double*>(sm_raw);  // [nb] values in descending order (gamma rule)
  float* p = reinterpret_cast<float*>(sorted + nb);    // [nb]
  int* ranks = reinterpret_cast<int*>(p + nb);         // [nb]
  uint8_t* sel = reinterpret_cast<uint8_t*>(ranks + nb);  // [nb]
  __shared__ float fscratch[32];
  __shared__ int iscratch[32];
  __shared__ int s_k;
  __shared__ float s_med[2];
  const int h = blockIdx.x, dir = blockIdx.y, tid = threadIdx.x;
  uint32_t* out = dir == 0 ? w.selv + static_cast<size_t>(h) * w.words
                           : w.selsr + static_cast<size_t>(h) * (w.words + 2);
  const int out_words = dir == 0 ? w.words : w.words + 2;
  if (pattern[h] != CRISP_PATTERN_VS) {
    for (int i = tid; i < out_words; i += blockDim.x) out[i] = 0u;
    return;
  }
  const float* src = (dir == 0 ? p_v : p_s) + static_cast<size_t>(h) * nb;
  for (int i = tid; i < nb; i += blockDim.x) p[i] = src[i];
  __syncthreads();

  bool need_rank = false;
  int k = nb;
  float thr = -1.f;  // N_b <= 2: every block is kept
  if (nb > 2) {
    // noise floor over the blocks that are not always retained (Eq. 3), as the sum of the middle blocks
    float part = 0.f;
    for (int i = 1 + tid; i < nb - 1; i += blockDim.x) part += p[i];
    const float r = block_sum<float>(part, fscratch);
    float mu = r / static_cast<float>(nb - 2);
    if (d.selector == 2) {
      // median of the middle blocks instead of their mean (Appendix H): the two central order statistics
      // are found by ranking the middle blocks among themselves
      const int n_mid = nb - 2;
      const int lo_rank = n_mid - 1 - (n_mid - 1) / 2, hi_rank = n_mid - 1 - n_mid / 2;  // descending ranks
      for (int e = 1 + tid; e < nb - 1; e += blockDim.x) {
        const float pe = p[e];
        int rank = 0;
        for (int j = 1; j < nb - 1; ++j) {
          const float pj = p[j];
          rank += (pj > pe || (pj == pe && j < e)) ? 1 : 0;
        }
        if (rank == lo_rank) s_med[0] = pe;
        if (rank == hi_rank) s_med[1] = pe;
      }
      __syncthreads();
      mu = 0.5f * (s_med[0] + s_med[1]);
    }
    thr = d.alpha * mu;
    if (d.selector == 0 || d.selector == 2) {
      int c = 0;
      for (int i = tid; i < nb; i += blockDim.x) c += (p[i] > thr) ? 1 : 0;
      const int cnt = block_sum<int>(c, iscratch);
      if (cnt >= d.k_min) {
        k = cnt;  // the top-cnt set is exactly {p > thr} (Eq. 4)
      } else {
        k = min(d.k_min, nb);
        need_rank = true;
      }
    } else {
      need_rank = true;
    }
  }
  if (!need_rank) {
    for (int i = tid; i < nb; i += blockDim.x) sel[i] = p[i] > thr;
  } else {
    // rank in the stable descending order: larger value first, then lower index
    for (int e = tid; e < nb; e += blockDim.x) {
      const float pe = p[e];
      int rank = 0;
      for (int j = 0; j < nb; ++j) {
        const float pj = p[j];
        rank += (pj > pe || (pj == pe && j < e)) ? 1 : 0;
      }
      ranks[e] = rank;
      sorted[rank] = static_cast<double>(pe);
    }
    __syncthreads();
    if (d.selector == 1) {
      // smallest k whose running sum (in sorted order) reaches gamma (Algorithm 6); all if never
      if (tid == 0) {
        double c = 0.0;
        int found = nb;
        for (int i = 0; i < nb; ++i) {
          c += sorted[i];
          if (c >= static_cast<double>(d.gamma)) {
            found = i + 1;
            break;
          }
        }
        s_k = min(max(found, d.k_min), nb);
      }
      __syncthreads();
      k = s_k;
    }
    for (int e = tid; e < nb; e += blockDim.x) sel[e] = ranks[e] < k;
  }
  __syncthreads();
  // bitmaps: vertical as is; slash reversed (bit x <-> offset nb-1-x) and zero padded
  for (int wd = tid; wd < out_words; wd += blockDim.x) {
    uint32_t bits = 0;
    for (int b = 0; b < 32; ++b) {
      const int x = wd * 32 + b;
      if (x < nb) {
        const int e = dir == 0 ? x : nb - 1 - x;
        bits |= static_cast<uint32_t>(sel[e] != 0) << b;
      }
    }
    out[wd] = bits;
  }
}

// ------------------------------------------------------------------------------------------------
// PE heads: pooling, pooled logits, row softmax
// ------------------------------------------------------------------------------------------------
// Block means of one [128 tokens, 128 dims] tile per CTA.  x is [n, heads, 128] bf16.
__global__ void __launch_bounds__(128)
pool_kernel(const Dims d, const __nv_bfloat16* __restrict__ x, int heads, int is_query,
            const int32_t* __restrict__ pattern, float* __restrict__ out, __nv_bfloat16* __restrict__ split) {
  const int J = blockIdx.x, h = blockIdx.y, tid = threadIdx.x;
  if (pattern == nullptr) {
    // comparison router: every head's block means are wanted
  } else if (is_query) {
    if (pattern[h] != CRISP_PATTERN_PE) return;
  } else {
    bool any = false;
    for (int g = 0; g < d.group; ++g) any = any || (pattern[h * d.group + g] == CRISP_PATTERN_PE);
    if (!any) return;
  }
  const int pair = tid & 63, half = tid >> 6;
  const __nv_bfloat162* base = reinterpret_cast<const __nv_bfloat162*>(
      x + (static_cast<size_t>(J) * kBlock + half * 64) * heads * kHeadDim + static_cast<size_t>(h) * kHeadDim);
  float a0 = 0.f, a1 = 0.f;
  // the last block may hold fewer than 128 tokens: rows at or beyond n are not read
  const int valid = min(kBlock, d.n - J * kBlock);
  const int rows = min(max(valid - half * 64, 0), 64);
  if (rows == 64) {
    // full half block: a fixed trip count keeps all 64 loads of a thread in flight
#pragma unroll
    for (int t = 0; t < 64; ++t) {
      const float2 v = __bfloat1622float2(base[static_cast<size_t>(t) * heads * (kHeadDim / 2) + pair]);
      a0 += v.x;
      a1 += v.y;
    }
  } else {
    for (int t = 0; t < rows; ++t) {
      const float2 v = __bfloat1622float2(base[static_cast<size_t>(t) * heads * (kHeadDim / 2) + pair]);
      a0 += v.x;
      a1 += v.y;
    }
  }
  __shared__ float2 other[64];
  if (half == 1) other[pair] = make_float2(a0, a1);
  __syncthreads();
  if (half == 0) {
    float* o = out + (static_cast<size_t>(h) * d.nb + J) * kHeadDim;
    const float inv = 1.0f / static_cast<float>(valid);
    const float m0 = (a0 + other[pair].x) * inv, m1 = (a1 + other[pair].y) * inv;
    o[2 * pair] = m0;
    o[2 * pair + 1] = m1;
    if (split != nullptr) {
      // mean = hi + mid + lo with three bf16 terms (the remainders are exact in fp32): the pooled logits are
      // then a sum of bf16 tensor-core products that reproduces the fp32 product to ~2^-24
      float r0 = m0, r1 = m1;
#pragma unroll
      for (int pl = 0; pl < 3; ++pl) {
        const __nv_bfloat162 t = __floats2bfloat162_rn(r0, r1);
        reinterpret_cast<__nv_bfloat162*>(split + ((static_cast<size_t>(pl) * d.nb + J) * heads + h) * kHeadDim)[pair] = t;
        r0 -= __low2float(t);
        r1 -= __high2float(t);
      }
    }
  }
}

// Pooled logits Z[m, J] = qbar[m] . kbar[J] * scale_log2, one 128 x 128 tile of (query block, key block) pairs per
// CTA, on the tensor cores.  The selection compares these values, so bf16 operands alone would not do: each fp32
// block mean is split into three bf16 terms (pool_kernel), and the six products hi*hi, hi*mid, mid*hi, mid*mid,
// hi*lo, lo*hi - accumulated in fp32 in TMEM, smallest first - reproduce the fp32 dot product to ~2^-24.
struct LogitsMaps {
  CUtensorMap q[3], k[3];
};
struct LogitsSmem {
  alignas(1024) uint8_t a[3][2][16384];  // [term][64-dim half] 128 block means of Q, 128-byte swizzle
  alignas(1024) uint8_t b[3][2][16384];  // the same for K
  uint64_t bar_in, bar_mma;
  uint32_t tmem_base;
  int abort_flag;
};

__global__ void __launch_bounds__(160)
pe_logits_kernel(const __grid_constant__ LogitsMaps maps, const Dims d, const int32_t* __restrict__ pattern,
                 const SelectPtrs w, int* status) {
  const int jt = blockIdx.x, mt = blockIdx.y, h = blockIdx.z;
  if (jt > mt || pattern[h] != CRISP_PATTERN_PE) return;
  extern __shared__ uint8_t smem_raw[];
  LogitsSmem& s = *reinterpret_cast<LogitsSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    s.abort_flag = 0;
    mbar_init(&s.bar_in, 1);
    mbar_init(&s.bar_mma, 1);
    fence_mbar_init();
  }
  if (warp == 4) {
    tmem_alloc(&s.tmem_base, 128);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tm = s.tmem_base;
  bool ok = true;
  if (warp == 4) {
    if (lane == 0) {
      mbar_arrive_expect_tx(&s.bar_in, 6u * 32768u);
      for (int pl = 0; pl < 3; ++pl) {
        tma_load_3d(s.a[pl][0], &maps.q[pl], &s.bar_in, 0, h, mt * kBlock);
        tma_load_3d(s.a[pl][1], &maps.q[pl], &s.bar_in, 64, h, mt * kBlock);
        tma_load_3d(s.b[pl][0], &maps.k[pl], &s.bar_in, 0, h / d.group, jt * kBlock);
        tma_load_3d(s.b[pl][1], &maps.k[pl], &s.bar_in, 64, h / d.group, jt * kBlock);
      }
      ok = mbar_wait(&s.bar_in, 0, &s.abort_flag);
      if (ok) {
        tc_fence_after_sync();
        constexpr uint32_t idesc = umma_idesc_bf16(128, 128, false, false);
        // (term of Q, term of K), smallest products first
        const int pa[6] = {2, 0, 1, 1, 0, 0}, pb[6] = {0, 2, 1, 0, 1, 0};
#pragma unroll
        for (int t = 0; t < 6; ++t)
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint64_t ad = umma_desc_sw128(smem_u32(s.a[pa[t]][kk >> 2]) + (kk & 3) * 32, 0, 1024);
            const uint64_t bd = umma_desc_sw128(smem_u32(s.b[pb[t]][kk >> 2]) + (kk & 3) * 32, 0, 1024);
            umma_ss(tm, ad, bd, idesc, (t > 0 || kk > 0) ? 1u : 0u);
          }
        umma_commit(&s.bar_mma);
      }
    }
    __syncwarp();
  } else {
    // ---- one thread per row of the tile: scale, then through shared memory so that the rows go out coalesced
    ok = mbar_wait(&s.bar_mma, 0, &s.abort_flag);
    float* stage = reinterpret_cast<float*>(s.a);  // 128 x 129 floats over the operand tiles, which are dead now
    if (ok) {
      tc_fence_after_sync();
      const uint32_t lane_addr = static_cast<uint32_t>(warp * 32) << 16;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        tmem_ld_x32(tm + lane_addr + c * 32, r);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) stage[tid * 129 + c * 32 + i] = __uint_as_float(r[i]) * d.scale_log2;
      }
    }
    named_bar_sync(1, 128);
    if (ok) {
      float* am = w.amat + static_cast<size_t>(h) * d.nb * d.nb;
      for (int rr = warp; rr < kBlock; rr += 4) {
        const int m = mt * kBlock + rr;
        if (m >= d.nb) break;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int J = jt * kBlock + c * 32 + lane;
          if (J <= m) am[static_cast<size_t>(m) * d.nb + J] = stage[rr * 129 + c * 32 + lane];
        }
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (tid == 0 && s.abort_flag) atomicExch(status, CRISP_ERR_DEVICE_TIMEOUT);
  if (warp == 4) tmem_dealloc(tm, 128);
}

// Row softmax over J <= m, divided by N_b (= the total of the pooled map).
__global__ void __launch_bounds__(256)
pe_normalise_kernel(const Dims d, const int32_t* __restrict__ pattern, const SelectPtrs w) {
  const int m = blockIdx.x, h = blockIdx.y, tid = threadIdx.x;
  if (pattern[h] != CRISP_PATTERN_PE) return;
  float* row = w.amat + (static_cast<size_t>(h) * d.nb + m) * d.nb;
  __shared__ float red[32];
  __shared__ float fscratch[32];
  float mx = -INFINITY;
  for (int J = tid; J <= m; J += 256) mx = fmaxf(mx, row[J]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if ((tid & 31) == 0) red[tid >> 5] = mx;
  __syncthreads();
  mx = red[0];
  for (int i = 1; i < 8; ++i) mx = fmaxf(mx, red[i]);
  float sum = 0.f;
  for (int J = tid; J <= m; J += 256) sum += exp2f(row[J] - mx);
  const float total = block_sum<float>(sum, fscratch);
  const float inv = 1.0f / (total * static_cast<float>(d.nb));
  for (int J = tid; J <= m; J += 256) row[J] = exp2f(row[J] - mx) * inv;
}

// ------------------------------------------------------------------------------------------------
// PE heads: gamma cut by radix histogram over the value bits
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ bool key_in_level(unsigned int key, unsigned int prefix, int level, int* bin) {
  if (level == 0) {
    *bin = static_cast<int>(key >> 20);
    return true;
  }
  if (level == 1) {
    *bin = static_cast<int>((key >> 9) & 2047u);
    return (key >> 20) == (prefix >> 20);
  }
  *bin = static_cast<int>(key & 511u);
  return (key >> 9) == (prefix >> 9);
}

__global__ void __launch_bounds__(256)
pe_hist_kernel(const Dims d, const int32_t* __restrict__ pattern, const SelectPtrs w, int level) {
  const int h = blockIdx.y, tid = threadIdx.x;
  if (pattern[h] != CRISP_PATTERN_PE) return;
  __shared__ unsigned int cnt[2048];
  __shared__ unsigned long long mass[2048];
  const int nbins = level == 2 ? kL2Bins : 2048;
  for (int i = tid; i < nbins; i += 256) {
    cnt[i] = 0u;
    mass[i] = 0ull;
  }
  __syncthreads();
  const unsigned int prefix = w.cut[h].prefix;
  if (level > 0 && w.cut[h].take == -1) return;  // gamma is out of reach: everything is kept
  const float* am = w.amat + static_cast<size_t>(h) * d.nb * d.nb;
  for (int m = blockIdx.x; m < d.nb; m += gridDim.x) {
    const float* row = am + static_cast<size_t>(m) * d.nb;
    // 1024 entries per pass: the four loads of a thread are issued before any of them is binned
    for (int J0 = 0; J0 <= m; J0 += 1024) {
      float vals[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int J = J0 + 256 * u + tid;
        vals[u] = J <= m ? row[J] : 0.f;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int J = J0 + 256 * u + tid;
        if (J0 + 256 * u > m) break;  // uniform: the whole chunk lies beyond the row
        int bin = -1;
        unsigned long long fixed = 0ull;
        if (J <= m) {
          const float v = vals[u];
          int b;
          if (key_in_level(__float_as_uint(v), prefix, level, &b)) {
            bin = b;
            fixed = __float2ull_rn(v * kMassScale);
          }
        }
        // Level 0: neighbouring entries of a flat map fall into a handful of bins: lanes with the same bin elect a
        // leader and add their counts and masses (three 20-bit limbs, summed exactly) in one atomic each.
        if (level > 0) {
          // lower levels: the 11 / 9 bits below the fixed prefix spread the entries over many bins
          if (bin >= 0) {
            atomicAdd(&cnt[bin], 1u);
            atomicAdd(&mass[bin], fixed);
          }
          continue;
        }
        const unsigned int peers = __match_any_sync(0xffffffffu, bin);
        const unsigned int l0 = __reduce_add_sync(peers, static_cast<unsigned int>(fixed & 0xFFFFFull));
        const unsigned int l1 = __reduce_add_sync(peers, static_cast<unsigned int>((fixed >> 20) & 0xFFFFFull));
        const unsigned int l2 = __reduce_add_sync(peers, static_cast<unsigned int>(fixed >> 40));
        if (bin >= 0 && (tid & 31) == __ffs(peers) - 1) {
          atomicAdd(&cnt[bin], static_cast<unsigned int>(__popc(peers)));
          atomicAdd(&mass[bin], static_cast<unsigned long long>(l0) + (static_cast<unsigned long long>(l1) << 20) +
                                    (static_cast<unsigned long long>(l2) << 40));
        }
      }
    }
  }
  __syncthreads();
  const int off = level == 0 ? 0 : (level == 1 ? kL0Bins : kL0Bins + kL1Bins);
  unsigned int* gc = w.hcount + static_cast<size_t>(h) * kHistStride + off;
  unsigned long long* gm = w.hmass + static_cast<size_t>(h) * kHistStride + off;
  for (int i = tid; i < nbins; i += 256)
    if (cnt[i]) {
      atomicAdd(&gc[i], cnt[i]);
      atomicAdd(&gm[i], mass[i]);
    }
}

// One CTA per head: the bins are read once, in parallel (two per thread, largest values first), an exclusive
// block scan gives the mass above every bin, and the first non-empty bin at which the mass reaches gamma
// is the one the cut falls into.
__global__ void __launch_bounds__(1024)
pe_cut_kernel(const Dims d, const int32_t* __restrict__ pattern, const SelectPtrs w, int level) {
  const int h = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (pattern[h] != CRISP_PATTERN_PE) return;
  const int nbins = level == 2 ? kL2Bins : 2048;
  const int off = level == 0 ? 0 : (level == 1 ? kL0Bins : kL0Bins + kL1Bins);
  const unsigned int* gc = w.hcount + static_cast<size_t>(h) * kHistStride + off;
  const unsigned long long* gm = w.hmass + static_cast<size_t>(h) * kHistStride + off;
  CutState c = w.cut[h];
  if (level == 0) {
    c.prefix = 0u;
    c.mass_above = 0ull;
    c.cutkey = 0u;
    c.take = 0x7fffffffffffffffLL;
  } else if (c.take == -1) {  // gamma was never reached at an earlier level: everything is kept
    return;
  }
  const double gd = static_cast<double>(d.gamma) * static_cast<double>(kMassScale);
  const unsigned long long gamma = gd >= 1.8e19 ? 0xffffffffffffffffull : static_cast<unsigned long long>(gd);

  // position p (0 = largest values) is bin nbins - 1 - p; thread t owns positions 2t and 2t + 1
  const int p0 = 2 * tid, p1 = 2 * tid + 1;
  const unsigned long long m0 = p0 < nbins ? gm[nbins - 1 - p0] : 0ull, m1 = p1 < nbins ? gm[nbins - 1 - p1] : 0ull;
  const unsigned int c0 = p0 < nbins ? gc[nbins - 1 - p0] : 0u, c1 = p1 < nbins ? gc[nbins - 1 - p1] : 0u;
  // exclusive scan of the per-thread sums: warp shuffles, then the 32 warp totals
  __shared__ unsigned long long warp_tot[32];
  __shared__ int first_hit;
  __shared__ unsigned long long total_mass;
  if (tid == 0) first_hit = 0x7fffffff;
  const unsigned long long mine = m0 + m1;
  unsigned long long incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const unsigned long long wt = warp_tot[lane];
    unsigned long long wi = wt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long t = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += t;
    }
    warp_tot[lane] = wi - wt;  // mass of the warps before this one
    if (lane == 31) total_mass = wi;
  }
  __syncthreads();
  const unsigned long long before0 = c.mass_above + warp_tot[warp] + (incl - mine);  // mass above position p0
  const unsigned long long before1 = before0 + m0;
  const bool hit0 = c0 != 0u && before0 + m0 >= gamma, hit1 = c1 != 0u && before1 + m1 >= gamma;
  if (hit0 || hit1) atomicMin(&first_hit, hit0 ? p0 : p1);
  __syncthreads();
  const int fp = first_hit;
  if (fp == 0x7fffffff) {
    if (tid == 0) {
      // the target exceeds the total mass (gamma >= 1 or rounding): keep every causal entry
      c.cutkey = 0u;
      c.take = -1;
      c.mass_above += total_mass;
      w.cut[h] = c;
    }
    return;
  }
  if (fp != p0 && fp != p1) return;
  // the thread that owns the bin of the cut finishes the level
  const int found = nbins - 1 - fp;
  const unsigned long long above = fp == p0 ? before0 : before1;
  const unsigned int found_count = fp == p0 ? c0 : c1;
  c.mass_above = above;
  const int shift = level == 0 ? 20 : (level == 1 ? 9 : 0);
  c.prefix |= static_cast<unsigned int>(found) << shift;
  if (level == 2) {
    c.cutkey = c.prefix;
    // all entries of this bin are equal; t = the smallest count whose mass reaches gamma
    const unsigned long long v = __float2ull_rn(__uint_as_float(c.cutkey) * kMassScale);
    long long t = 1;
    if (v > 0ull) {
      const unsigned long long need = gamma - above;  // > 0 here
      t = static_cast<long long>((need + v - 1ull) / v);
    }
    if (t < 1) t = 1;
    if (t > static_cast<long long>(found_count)) t = static_cast<long long>(found_count);
    c.take = t;
  }
  w.cut[h] = c;
}

// Per row of a PE head: how many entries lie above the cut, how many tie with it, and how the two
// forced entries (column 0 and the diagonal) compare.
__global__ void __launch_bounds__(256)
pe_row_stats_kernel(const Dims d, const int32_t* __restrict__ pattern, const SelectPtrs w) {
  const int m = blockIdx.x, h = blockIdx.y, tid = threadIdx.x;
  if (pattern[h] != CRISP_PATTERN_PE) return;
  __shared__ int iscratch[32];
  const CutState c = w.cut[h];
  const float* row = w.amat + (static_cast<size_t>(h) * d.nb + m) * d.nb;
  int gt = 0, eq = 0;
  for (int J = tid; J <= m; J += 256) {
    const unsigned int key = __float_as_uint(row[J]);
    gt += key > c.cutkey;
    eq += key == c.cutkey;
  }
  gt = block_sum<int>(gt, iscratch);
  eq = block_sum<int>(eq, iscratch);
  if (tid == 0) {
    const unsigned int k0 = __float_as_uint(row[0]), km = __float_as_uint(row[m]);
    const int f = (k0 > c.cutkey ? 1 : 0) | (k0 == c.cutkey ? 2 : 0) | (km > c.cutkey ? 4 : 0) |
                  (km == c.cutkey ? 8 : 0);
    const size_t o = static_cast<size_t>(h) * d.nb + m;
    w.n_gt[o] = gt;
    w.n_eq[o] = eq;
    w.flags[o] = f;
  }
}

// Per PE head: ties are taken in row-major order, so row m takes clamp(T - (ties in rows < m), 0, ties_m).
__global__ void __launch_bounds__(1024)
pe_take_kernel(const Dims d, const int32_t* __restrict__ pattern, const SelectPtrs w) {
  const int h = blockIdx.x, tid = threadIdx.x;
  if (pattern[h] != CRISP_PATTERN_PE) return;
  __shared__ long long scratch[33];
  const int seg = (d.nb + 1023) / 1024;
  const int b0 = min(tid * seg, d.nb), b1 = min(b0 + seg, d.nb);
  const size_t base = static_cast<size_t>(h) * d.nb;
  long long local = 0;
  for (int m = b0; m < b1; ++m) local += w.n_eq[base + m];
  long long before = block_exclusive_scan_1024(local, scratch, nullptr);
  const CutState c = w.cut[h];
  for (int m = b0; m < b1; ++m) {
    const int eq = w.n_eq[base + m];
    int take;
    if (c.take < 0) {
      take = eq;
    } else {
      const long long left = c.take - before;
      take = static_cast<int>(left <= 0 ? 0 : (left >= eq ? eq : left));
    }
    before += eq;
    const int f = w.flags[base + m];
    const bool sel0 = (f & 1) || ((f & 2) && take >= 1);
    const bool selm = (f & 4) || ((f & 8) && take >= eq);
    int count = w.n_gt[base + m] + take + (sel0 ? 0 : 1);
    if (m > 0) count += selm ? 0 : 1;
    w.take[base + m] = take;
    w.counts[base + m] = count;
  }
}

// ------------------------------------------------------------------------------------------------
// Expansion of VS heads, row lengths, scan, fill
// ------------------------------------------------------------------------------------------------
// Word `wd` (key blocks 32*wd .. 32*wd+31) of the keep bitmap of query block m of a VS head.
__device__ __forceinline__ uint32_t vs_keep_word(const uint32_t* __restrict__ selv, const uint32_t* __restrict__ selsr,
                                                 int nb, int m, int wd) {
  const int sh = nb - 1 - m;              // slash offset s = m - J  <->  reversed bit J + sh
  const int pos0 = wd * 32 + sh, pos1 = pos0 + 1;
  const uint32_t a = __funnelshift_r(selsr[pos0 >> 5], selsr[(pos0 >> 5) + 1], pos0 & 31);
  const uint32_t b = __funnelshift_r(selsr[pos1 >> 5], selsr[(pos1 >> 5) + 1], pos1 & 31);
  uint32_t bits = selv[wd] | a | b;
  if (wd == 0) bits |= 1u;
  if (wd == (m >> 5)) {
    bits |= 1u << (m & 31);
    const int top = m & 31;
    bits &= (top == 31) ? 0xffffffffu : ((2u << top) - 1u);
  }
  return bits;
}

__global__ void __launch_bounds__(256)
count_vs_kernel(const Dims d, const int32_t* __restrict__ pattern, const SelectPtrs w) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m = blockIdx.x * 8 + warp, h = blockIdx.y;
  if (m >= d.nb || pattern[h] != CRISP_PATTERN_VS) return;
  const uint32_t* selv = w.selv + static_cast<size_t>(h) * w.words;
  const uint32_t* selsr = w.selsr + static_cast<size_t>(h) * (w.words + 2);
  int c = 0;
  for (int wd = lane; wd <= (m >> 5); wd += 32) c += __popc(vs_keep_word(selv, selsr, d.nb, m, wd));
  c = warp_sum_i(c);
  if (lane == 0) w.counts[static_cast<size_t>(h) * d.nb + m] = c;
}

// Exclusive scan of all row lengths (head-major) into row_ptr; total into *nnz_needed; capacity check.
__global__ void __launch_bounds__(1024)
scan_rows_kernel(const Dims d, const SelectPtrs w, int64_t* __restrict__ row_ptr, int64_t capacity,
                 int64_t* __restrict__ nnz_needed, int* status) {
  const int tid = threadIdx.x;
  const long long total_rows = static_cast<long long>(d.hq) * d.nb;
  __shared__ long long scratch[33];
  long long carry = 0;
  // 4096 consecutive rows per pass, four per thread (coalesced), scanned across the block
  for (long long base = 0; base < total_rows; base += 4096) {
    const long long r0 = base + 4 * tid;
    int c[4];
    long long local = 0;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      c[u] = r0 + u < total_rows ? w.counts[r0 + u] : 0;
      local += c[u];
    }
    long long pass_total;
    long long run = carry + block_exclusive_scan_1024(local, scratch, &pass_total);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const long long r = r0 + u;
      if (r < total_rows) {
        const int h = static_cast<int>(r / d.nb), m = static_cast<int>(r % d.nb);
        row_ptr[static_cast<size_t>(h) * (d.nb + 1) + m] = run;
        run += c[u];
        if (m == d.nb - 1) row_ptr[static_cast<size_t>(h) * (d.nb + 1) + d.nb] = run;
      }
    }
    carry += pass_total;
  }
  if (tid == 0) {
    *nnz_needed = carry;
    if (carry > capacity) atomicExch(status, CRISP_ERR_CAPACITY);
  }
}

__global__ void __launch_bounds__(256)
fill_kernel(const Dims d, const int32_t* __restrict__ pattern, const SelectPtrs w,
            const int64_t* __restrict__ row_ptr, int32_t* __restrict__ col_idx, int64_t capacity,
            const int64_t* __restrict__ nnz_needed) {
  if (*nnz_needed > capacity) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m = blockIdx.x * 8 + warp, h = blockIdx.y;
  if (m >= d.nb) return;
  int32_t* out = col_idx + row_ptr[static_cast<size_t>(h) * (d.nb + 1) + m];
  int written = 0;
  if (pattern[h] == CRISP_PATTERN_VS) {
    const uint32_t* selv = w.selv + static_cast<size_t>(h) * w.words;
    const uint32_t* selsr = w.selsr + static_cast<size_t>(h) * (w.words + 2);
    const int nwords = (m >> 5) + 1;
    for (int w0 = 0; w0 < nwords; w0 += 32) {
      const int wd = w0 + lane;
      uint32_t bits = wd < nwords ? vs_keep_word(selv, selsr, d.nb, m, wd) : 0u;
      const int c = __popc(bits);
      int incl = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      // emit word by word, lane b owning bit b: the entries of a word go out as one contiguous store
      const int nw = min(32, nwords - w0);
      for (int k = 0; k < nw; ++k) {
        const uint32_t wbits = __shfl_sync(0xffffffffu, bits, k);
        if (wbits == 0u) continue;
        const int base = written + __shfl_sync(0xffffffffu, incl - c, k);
        if ((wbits >> lane) & 1u) out[base + __popc(wbits & ((1u << lane) - 1u))] = (w0 + k) * 32 + lane;
      }
      written += __shfl_sync(0xffffffffu, incl, 31);
    }
  } else {
    const CutState c = w.cut[h];
    const float* row = w.amat + (static_cast<size_t>(h) * d.nb + m) * d.nb;
    const int take = w.take[static_cast<size_t>(h) * d.nb + m];
    int ties_seen = 0;
    // 128 columns per pass: the four loads of a lane are issued before the (serial) bookkeeping of the pass
    for (int J0 = 0; J0 <= m; J0 += 128) {
      unsigned int key[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int J = J0 + 32 * u + lane;
        key[u] = J <= m ? __float_as_uint(row[J]) : 0u;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int J = J0 + 32 * u + lane;
        const bool in = J <= m;
        const bool gt = in && key[u] > c.cutkey, eq = in && key[u] == c.cutkey;
        const uint32_t eqmask = __ballot_sync(0xffffffffu, eq);
        const int my_tie = ties_seen + __popc(eqmask & ((1u << lane) - 1u));
        const bool keep = in && (gt || (eq && my_tie < take) || J == 0 || J == m);
        const uint32_t keepmask = __ballot_sync(0xffffffffu, keep);
        if (keep) out[written + __popc(keepmask & ((1u << lane) - 1u))] = J;
        written += __popc(keepmask);
        ties_seen += __popc(eqmask);
      }
    }
  }
}

SelectPtrs carve(const Dims& d, void* ws, size_t* total) {
  SelectPtrs w;
  uint8_t* base = static_cast<uint8_t*>(ws);
  size_t off = kWsHeader;
  auto take = [&](size_t bytes) {
    void* r = base + off;
    off += align_up(bytes, 256);
    return r;
  };
  w.words = (d.nb + 31) / 32;
  w.selv = static_cast<uint32_t*>(take(sizeof(uint32_t) * d.hq * w.words));
  w.selsr = static_cast<uint32_t*>(take(sizeof(uint32_t) * d.hq * (w.words + 2)));
  w.kbar = static_cast<float*>(take(sizeof(float) * d.hkv * d.nb * kHeadDim));
  w.qbar = static_cast<float*>(take(sizeof(float) * static_cast<size_t>(d.hq) * d.nb * kHeadDim));
  w.ksplit = static_cast<__nv_bfloat16*>(take(sizeof(__nv_bfloat16) * 3 * static_cast<size_t>(d.hkv) * d.nb * kHeadDim));
  w.qsplit = static_cast<__nv_bfloat16*>(take(sizeof(__nv_bfloat16) * 3 * static_cast<size_t>(d.hq) * d.nb * kHeadDim));
  w.amat = static_cast<float*>(take(sizeof(float) * static_cast<size_t>(d.hq) * d.nb * d.nb));
  w.hcount = static_cast<unsigned int*>(take(sizeof(unsigned int) * d.hq * kHistStride));
  w.hmass = static_cast<unsigned long long*>(take(sizeof(unsigned long long) * d.hq * kHistStride));
  w.cut = static_cast<CutState*>(take(sizeof(CutState) * d.hq));
  w.n_gt = static_cast<int*>(take(sizeof(int) * d.hq * d.nb));
  w.n_eq = static_cast<int*>(take(sizeof(int) * d.hq * d.nb));
  w.flags = static_cast<int*>(take(sizeof(int) * d.hq * d.nb));
  w.take = static_cast<int*>(take(sizeof(int) * d.hq * d.nb));
  w.counts = static_cast<int*>(take(sizeof(int) * d.hq * d.nb));
  *total = off;
  return w;
}

}  // namespace

size_t select_ws_bytes(const Dims& d) {
  size_t total;
  carve(d, nullptr, &total);
  return total;
}

int launch_select(const Dims& d, const void* q, const void* k, const int32_t* pattern, const float* p_v,
                  const float* p_s, void* ws, int64_t* row_ptr, int32_t* col_idx, int64_t capacity,
                  int64_t* nnz_needed, cudaStream_t stream) {
  if (d.nb > 8192) return CRISP_ERR_UNSUPPORTED;
  size_t total;
  SelectPtrs w = carve(d, ws, &total);
  int* status = static_cast<int*>(ws);
  CRISP_CUDA_TRY(cudaMemsetAsync(ws, 0, kWsHeader, stream), "select: clear status");
  CRISP_CUDA_TRY(cudaMemsetAsync(w.hcount, 0, sizeof(unsigned int) * d.hq * kHistStride, stream), "select: clear");
  CRISP_CUDA_TRY(cudaMemsetAsync(w.hmass, 0, sizeof(unsigned long long) * d.hq * kHistStride, stream), "select: clear");

  // VS heads
  const size_t vs_smem = (sizeof(double) + sizeof(float) + sizeof(int) + 1) * static_cast<size_t>(d.nb) + 16;
  CRISP_CUDA_TRY(cudaFuncSetAttribute(select_vs_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      static_cast<int>(vs_smem)),
                 "select: smem attribute");
  CRISP_KERNEL("select_vs", stream, select_vs_kernel<<<dim3(d.hq, 2), 1024, vs_smem, stream>>>(d, pattern, p_v, p_s, w));

  // PE heads (every kernel returns at once for heads routed to VS)
  const __nv_bfloat16* qb = static_cast<const __nv_bfloat16*>(q);
  const __nv_bfloat16* kb = static_cast<const __nv_bfloat16*>(k);
  CRISP_KERNEL("pool_k", stream, pool_kernel<<<dim3(d.nb, d.hkv), 128, 0, stream>>>(d, kb, d.hkv, 0, pattern, w.kbar, w.ksplit));
  CRISP_KERNEL("pool_q", stream, pool_kernel<<<dim3(d.nb, d.hq), 128, 0, stream>>>(d, qb, d.hq, 1, pattern, w.qbar, w.qsplit));
  {
    LogitsMaps maps;
    for (int pl = 0; pl < 3; ++pl) {
      int rc = make_tmap_bf16_nhd(&maps.q[pl], w.qsplit + static_cast<size_t>(pl) * d.nb * d.hq * kHeadDim, d.nb, d.hq);
      if (rc != CRISP_OK) return rc;
      rc = make_tmap_bf16_nhd(&maps.k[pl], w.ksplit + static_cast<size_t>(pl) * d.nb * d.hkv * kHeadDim, d.nb, d.hkv);
      if (rc != CRISP_OK) return rc;
    }
    const size_t smem = sizeof(LogitsSmem) + 1024;
    CRISP_CUDA_TRY(cudaFuncSetAttribute(pe_logits_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(smem)),
                   "select: smem attribute");
    const int nt = (d.nb + kBlock - 1) / kBlock;
    CRISP_KERNEL("pe_logits", stream, pe_logits_kernel<<<dim3(nt, nt, d.hq), 160, smem, stream>>>(maps, d, pattern, w, status));
  }
  CRISP_KERNEL("pe_normalise", stream, pe_normalise_kernel<<<dim3(d.nb, d.hq), 256, 0, stream>>>(d, pattern, w));
  const int hist_ctas = d.nb < 128 ? d.nb : 128;
  for (int level = 0; level < 3; ++level) {
    CRISP_KERNEL("pe_hist", stream, pe_hist_kernel<<<dim3(hist_ctas, d.hq), 256, 0, stream>>>(d, pattern, w, level));
    CRISP_KERNEL("pe_cut", stream, pe_cut_kernel<<<d.hq, 1024, 0, stream>>>(d, pattern, w, level));
  }
  CRISP_KERNEL("pe_row_stats", stream, pe_row_stats_kernel<<<dim3(d.nb, d.hq), 256, 0, stream>>>(d, pattern, w));
  CRISP_KERNEL("pe_take", stream, pe_take_kernel<<<d.hq, 1024, 0, stream>>>(d, pattern, w));

  // expansion + compaction
  CRISP_KERNEL("count_vs", stream, count_vs_kernel<<<dim3((d.nb + 7) / 8, d.hq), 256, 0, stream>>>(d, pattern, w));
  CRISP_KERNEL("scan_rows", stream, scan_rows_kernel<<<1, 1024, 0, stream>>>(d, w, row_ptr, capacity, nnz_needed, status));
  CRISP_KERNEL("fill", stream, fill_kernel<<<dim3((d.nb + 7) / 8, d.hq), 256, 0, stream>>>(d, pattern, w, row_ptr, col_idx, capacity,
                                                              nnz_needed));
  CRISP_CUDA_TRY(cudaGetLastError(), "select: launch");
  return CRISP_OK;
}

// ------------------------------------------------------------------------------------------------
// Comparison router (Algorithm 5): Jensen-Shannon distance between the pooled estimate
//   a_bar = Softmax(pool(Q_hat) pool(K)^T / sqrt(d))      (one row over the N_b key blocks)
// and the per-query mean a_hat = sumpool(Softmax(Q_hat K^T / sqrt(d))) = p_v from crisp_route.
// ------------------------------------------------------------------------------------------------
namespace {
__global__ void __launch_bounds__(256)
jsd_kernel(const Dims d, const __nv_bfloat16* __restrict__ q, const float* __restrict__ kbar,
           const float* __restrict__ p_v, float tau_jsd, float* __restrict__ jsd, int32_t* __restrict__ pattern) {
  extern __shared__ float z[];  // [nb] pooled logits, then a_bar
  __shared__ float qbar[kHeadDim];
  __shared__ float fscratch[32];
  const int h = blockIdx.x, tid = threadIdx.x;
  // mean of the last block's queries: thread pair (dim pair, half of the rows)
  {
    const int pair = tid & 63, part = tid >> 6;  // 4 parts of 32 rows
    const __nv_bfloat162* base = reinterpret_cast<const __nv_bfloat162*>(
        q + (static_cast<size_t>(d.n - kBlock) + part * 32) * d.hq * kHeadDim + static_cast<size_t>(h) * kHeadDim);
    float a0 = 0.f, a1 = 0.f;
    for (int t = 0; t < 32; ++t) {
      const float2 v = __bfloat1622float2(base[static_cast<size_t>(t) * d.hq * (kHeadDim / 2) + pair]);
      a0 += v.x;
      a1 += v.y;
    }
    __shared__ float2 parts[4][64];
    parts[part][pair] = make_float2(a0, a1);
    __syncthreads();
    if (tid < 64) {
      float2 s0 = parts[0][tid];
      for (int pp = 1; pp < 4; ++pp) {
        s0.x += parts[pp][tid].x;
        s0.y += parts[pp][tid].y;
      }
      qbar[2 * tid] = s0.x * (1.0f / kBlock);
      qbar[2 * tid + 1] = s0.y * (1.0f / kBlock);
    }
    __syncthreads();
  }
  const float* kb = kbar + static_cast<size_t>(h / d.group) * d.nb * kHeadDim;
  float mx = -INFINITY;
  for (int J = tid; J < d.nb; J += 256) {
    const float* kr = kb + static_cast<size_t>(J) * kHeadDim;
    float acc = 0.f;
    for (int c = 0; c < kHeadDim; ++c) acc = fmaf(qbar[c], kr[c], acc);
    acc *= d.scale;
    z[J] = acc;
    mx = fmaxf(mx, acc);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  __shared__ float red[8];
  if ((tid & 31) == 0) red[tid >> 5] = mx;
  __syncthreads();
  mx = red[0];
  for (int i = 1; i < 8; ++i) mx = fmaxf(mx, red[i]);
  float sum = 0.f;
  for (int J = tid; J < d.nb; J += 256) {
    const float e = expf(z[J] - mx);
    z[J] = e;
    sum += e;
  }
  const float total = block_sum<float>(sum, fscratch);
  const float inv = 1.0f / total;
  // 0.5 KL(a_hat || m) + 0.5 KL(a_bar || m), m = (a_hat + a_bar) / 2; zero-probability terms contribute 0
  float acc = 0.f;
  const float* ah = p_v + static_cast<size_t>(h) * d.nb;
  for (int J = tid; J < d.nb; J += 256) {
    const float a = ah[J], b = z[J] * inv;
    const float m = 0.5f * (a + b);
    if (a > 0.f) acc += 0.5f * a * logf(a / m);
    if (b > 0.f) acc += 0.5f * b * logf(b / m);
  }
  const float js = block_sum<float>(acc, fscratch);
  if (tid == 0) {
    const float dist = sqrtf(fmaxf(js, 0.f));
    jsd[h] = dist;
    pattern[h] = dist >= tau_jsd ? CRISP_PATTERN_VS : CRISP_PATTERN_PE;
  }
}
}  // namespace

int launch_route_jsd(const Dims& d, const void* q, const void* k, const float* p_v, void* ws, float tau_jsd,
                     float* jsd, int32_t* pattern, cudaStream_t stream) {
  if (d.nb > 8192) return CRISP_ERR_UNSUPPORTED;
  size_t total;
  SelectPtrs w = carve(d, ws, &total);
  CRISP_CUDA_TRY(cudaMemsetAsync(ws, 0, kWsHeader, stream), "route_jsd: clear status");
  CRISP_KERNEL("pool_k", stream, pool_kernel<<<dim3(d.nb, d.hkv), 128, 0, stream>>>(d, static_cast<const __nv_bfloat16*>(k), d.hkv, 0, nullptr,
                                                     w.kbar, nullptr));
  CRISP_KERNEL("jsd", stream, jsd_kernel<<<d.hq, 256, sizeof(float) * d.nb, stream>>>(d, static_cast<const __nv_bfloat16*>(q), w.kbar, p_v,
                                                         tau_jsd, jsd, pattern));
  CRISP_CUDA_TRY(cudaGetLastError(), "route_jsd: launch");
  return CRISP_OK;
}

}  // namespace crisp
