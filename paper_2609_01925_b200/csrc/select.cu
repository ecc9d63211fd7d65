// Stage 3b-3c: block selection and expansion into per-query-block key-block lists.
//
//   VS heads  (Algorithm 3 lines 6-12 / Eq. 3-4; Algorithm 6 when selector == 1; the median floor of
//     Appendix H when selector == 2): `prepare_kernel`, one CTA per head, keeps p_d in shared memory,
//     computes the noise floor, the budget k_d and the top-k_d set (ties to the lower index) of both
//     directions as bitmaps, then the length of every query block's list (popcounts of the vertical
//     bitmap, the shifted slash bitmap and the forced blocks {0, m}) and their prefix sum inside the head.
//     The other CTAs of the same launch compute the block means of Q and K that the PE heads need.
//   PE heads  (Algorithm 4): pooled logits on the tensor cores (`pe_logits_kernel`), which also leaves the
//     row maximum and 1 / (row sum * N_b) of every row, so the causal row softmax divided by the total is
//     never written: every later pass recomputes an entry as 2^(z - max) * inv from the stored logit.  The
//     gamma cut is found WITHOUT a sort by a three-level radix histogram (8 + 12 + 11 bits) over the fp32 bit patterns of
//     those values (`pe_hist_kernel<level>`, masses in exact fixed point; the last CTA of a head to finish
//     a level locates the cut in it), which yields the value at the cut and how many entries tied with it
//     are taken (ties in row-major order).  The last level also counts, per row, the entries above the
//     cut's bin; `pe_rows_kernel` re-reads only the rows that have entries inside that bin, distributes the
//     ties and scans the row lengths of the head.
//   `fill_kernel` adds the heads' totals up to global offsets, writes row_ptr and the ascending column
//     lists.  No atomics touch the lists, and the histograms add integers, so everything is reproducible.
//
// Passes over the pooled map (4 N_b^2 / 2 bytes per PE head): one write (logits), three reads (histogram
// levels), one read (fill); rows holding entries in the cut's last bin are read once more (a few).
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace crisp {
using namespace sm100;

namespace {

// Radix levels over the fp32 bit pattern of a (positive) value: the exponent (key bits 30..23), then twelve and
// eleven mantissa bits (22..11, 10..0).  Level 0 sees every entry, and a row's entries share two or three
// exponents, so its few bins are fed through warp-wide sums; the lower levels see only the entries inside the
// cut's bin, spread over thousands of bins.
constexpr int kL0Bins = 256, kL1Bins = 4096, kL2Bins = 2048;
constexpr int kL0Shift = 23, kL1Shift = 11;
constexpr int kHistStride = kL0Bins + kL1Bins + kL2Bins;
constexpr int kHistThreads = 512;
constexpr int kMaxBins = 4096;
__host__ __device__ constexpr int level_bins(int level) { return level == 0 ? kL0Bins : (level == 1 ? kL1Bins : kL2Bins); }
__host__ __device__ constexpr int level_offset(int level) { return level == 0 ? 0 : (level == 1 ? kL0Bins : kL0Bins + kL1Bins); }
__host__ __device__ constexpr int level_shift(int level) { return level == 0 ? kL0Shift : (level == 1 ? kL1Shift : 0); }

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
  // ---- zeroed at the start of every call (one contiguous region)
  unsigned int* hcount;        // [hq][kHistStride]
  unsigned long long* hmass;   // [hq][kHistStride] fixed-point mass per bin
  int* hist_done;              // [3][hq] CTAs of a head that finished a histogram level
  int* rows_done;              // [hq]   CTAs of a head that finished pe_rows
  size_t zero_bytes;
  // ---- written before read
  uint32_t* selv;   // [hq][words] vertical bitmap
  uint32_t* selsr;  // [hq][words + 2] reversed slash bitmap: bit x = S_s contains N_b-1-x
  float* kbar;      // [hkv][nb][128]
  float* qbar;      // [hq][nb][128]
  __nv_bfloat16* ksplit;  // [3][nb][hkv][128] block means of K as three bf16 terms (hi + mid + lo = the fp32 mean)
  __nv_bfloat16* qsplit;  // [3][nb][hq][128]  the same for Q
  float* amat;      // [hq][nb][nb] pooled logits in base-2 units (row m uses columns 0..m)
  float* row_m;     // [hq][nb] row maximum of the pooled logits
  float* row_inv;   // [hq][nb] 1 / (sum_J 2^(z - max) * N_b)
  CutState* cut;    // [hq]
  int* n_gt;        // [hq][nb] entries above the cut (first: above the cut's last bin)
  int* n_eq;        // [hq][nb] entries inside the cut's last bin, then: entries tied with the cut
  int* counts;      // [hq][nb] row lengths
  int* take;        // [hq][nb] ties of row m that are selected
  int* local_off;   // [hq][nb] exclusive prefix sum of the row lengths inside the head
  long long* head_total;  // [hq] entries of the head's lists
  int* pe_list;     // [hq + 1] the PE heads in ascending order, then (at index hq) how many there are
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

// ------------------------------------------------------------------------------------------------
// First launch: CTAs [0, hq) select the blocks of the VS heads and size their lists; the remaining CTAs
// pool Q and K for the PE heads.
// ------------------------------------------------------------------------------------------------
// Block means of eight [128 tokens, 128 dims] tiles per CTA (128 threads per tile).  x is [n, heads, 128] bf16.
__device__ __forceinline__ void pool_tile(const Dims& d, const __nv_bfloat16* __restrict__ x, int heads, int J, int h,
                                          int tid, float* __restrict__ out, __nv_bfloat16* __restrict__ split,
                                          float2* other /* [64] shared */, int bar_id) {
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
  if (half == 1) other[pair] = make_float2(a0, a1);
  named_bar_sync(bar_id, 128);
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

// Budget and top-k of one direction of a VS head (Algorithm 3 / Algorithm 6 / Appendix H) as a bitmap.
__device__ void select_direction(const Dims& d, const float* __restrict__ src, int dir, uint32_t* __restrict__ out,
                                 int out_words, double* sorted, float* p, int* ranks, uint8_t* sel, float* fscratch,
                                 int* iscratch, int* s_k, float* s_med) {
  const int nb = d.nb, tid = threadIdx.x;
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
        *s_k = min(max(found, d.k_min), nb);
      }
      __syncthreads();
      k = *s_k;
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
  __syncthreads();
}

__global__ void __launch_bounds__(1024)
prepare_kernel(const Dims d, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
               const int32_t* __restrict__ pattern, const float* __restrict__ p_v, const float* __restrict__ p_s,
               const SelectPtrs w, int vs_ctas, int pool_all_k) {
  pdl_enter();
  extern __shared__ uint8_t sm_raw[];
  const int tid = threadIdx.x;
  if (static_cast<int>(blockIdx.x) >= vs_ctas) {
    // ---------------- pooling: eight (block, head) tiles per CTA; heads [0, hkv) are K, the rest Q
    __shared__ float2 other[8][64];
    const int sub = tid >> 7, t = tid & 127;
    const long long tile = (static_cast<long long>(blockIdx.x) - vs_ctas) * 8 + sub;
    const long long n_tiles = static_cast<long long>(d.nb) * (d.hkv + d.hq);
    if (tile >= n_tiles) return;  // whole 128-thread groups leave together
    const int hh = static_cast<int>(tile / d.nb), J = static_cast<int>(tile % d.nb);
    if (hh < d.hkv) {
      bool any = pool_all_k != 0;
      for (int g = 0; g < d.group && !any; ++g) any = pattern[hh * d.group + g] == CRISP_PATTERN_PE;
      if (!any) return;
      pool_tile(d, k, d.hkv, J, hh, t, w.kbar, w.ksplit, other[sub], 1 + sub);
    } else {
      const int h = hh - d.hkv;
      if (pattern == nullptr || pattern[h] != CRISP_PATTERN_PE) return;
      pool_tile(d, q, d.hq, J, h, t, w.qbar, w.qsplit, other[sub], 1 + sub);
    }
    return;
  }
  // ---------------- VS head: both directions, then the lengths of its lists
  const int h = blockIdx.x, nb = d.nb;
  if (h == 0 && tid < 32) {
    // the PE heads in ascending order, for the pooled-logits kernel's work items
    int n = 0;
    for (int h0 = 0; h0 < d.hq; h0 += 32) {
      const bool pe = h0 + tid < d.hq && pattern[h0 + tid] == CRISP_PATTERN_PE;
      const uint32_t mask = __ballot_sync(0xffffffffu, pe);
      if (pe) w.pe_list[n + __popc(mask & ((1u << tid) - 1u))] = h0 + tid;
      n += __popc(mask);
    }
    if (tid == 0) w.pe_list[d.hq] = n;
  }
  if (pattern[h] != CRISP_PATTERN_VS) return;
  double* sorted = reinterpret_cast<double*>(sm_raw);  // [nb] values in descending order (gamma rule)
  float* p = reinterpret_cast<float*>(sorted + nb);    // [nb]
  int* ranks = reinterpret_cast<int*>(p + nb);         // [nb]
  uint8_t* sel = reinterpret_cast<uint8_t*>(ranks + nb);  // [nb]
  __shared__ float fscratch[32];
  __shared__ int iscratch[32];
  __shared__ long long lscratch[33];
  __shared__ int s_k;
  __shared__ float s_med[2];
  uint32_t* selv = w.selv + static_cast<size_t>(h) * w.words;
  uint32_t* selsr = w.selsr + static_cast<size_t>(h) * (w.words + 2);
  select_direction(d, p_v + static_cast<size_t>(h) * nb, 0, selv, w.words, sorted, p, ranks, sel, fscratch, iscratch,
                   &s_k, s_med);
  select_direction(d, p_s + static_cast<size_t>(h) * nb, 1, selsr, w.words + 2, sorted, p, ranks, sel, fscratch,
                   iscratch, &s_k, s_med);
  // the bitmaps were written by this CTA; the barrier at the end of select_direction makes them visible to it
  const int seg = (nb + 1023) / 1024;
  const int b0 = min(tid * seg, nb), b1 = min(b0 + seg, nb);
  const size_t base = static_cast<size_t>(h) * nb;
  long long local = 0;
  for (int m = b0; m < b1; ++m) {
    int c = 0;
    for (int wd = 0; wd <= (m >> 5); ++wd) c += __popc(vs_keep_word(selv, selsr, nb, m, wd));
    w.counts[base + m] = c;
    local += c;
  }
  long long total;
  long long run = block_exclusive_scan_1024(local, lscratch, &total);
  for (int m = b0; m < b1; ++m) {
    w.local_off[base + m] = static_cast<int>(run);
    run += w.counts[base + m];
  }
  if (tid == 0) w.head_total[h] = total;
}

// ------------------------------------------------------------------------------------------------
// PE heads: pooled logits on the tensor cores
// ------------------------------------------------------------------------------------------------
// Z[m, J] = qbar[m] . kbar[J] * scale * log2(e).  The selection compares these values, so bf16 operands alone
// would not do: each fp32 block mean is split into three bf16 terms (pool_tile), and the six products hi*hi,
// hi*mid, mid*hi, mid*mid, hi*lo, lo*hi - accumulated in fp32 in TMEM - reproduce the fp32 dot product to ~2^-24.
//
// Persistent CTAs.  A work item is one PE head and one strip of 128 query blocks (rows m); the strip's three
// operand terms stay in shared memory while the CTA walks over the strip's key tiles jt = 0 .. mt.  The K-side
// operands arrive in two halves of 64 dims (two 48 KB slots), loaded by a thread of their own: a slot is refilled
// the moment the MMAs that read it have completed, while the other half's MMAs run (with the loads issued by the
// MMA thread, which sits in the tensor pipe's queue while it issues, every half arrived ~1700 cycles late).
// Two TMEM accumulators and two groups of four epilogue warps (one thread per row; group 0 drains the even tiles
// of an item, group 1 the odd ones) keep the MMAs of tile t + 1 running while tile t is drained.  A strip holds
// complete rows, so the epilogue threads carry the running maximum and sum of their row across their tiles and
// leave the row's softmax normalisers at the end of the item; the normalised map itself is never written.  The
// logits go to global memory through a 32 x 32 staging tile per warp, so that a store writes whole 128-byte
// lines of four rows instead of 16 bytes of 32 rows.
struct LogitsMaps {
  CUtensorMap q[3], k[3];
};
struct LogitsSmem {
  alignas(1024) uint8_t a[3][2][16384];  // [term][64-dim half] 128 block means of Q, 128-byte swizzle
  alignas(1024) uint8_t b[2][3][16384];  // [64-dim half = slot][term] 128 block means of K
  uint64_t bar_a_full, bar_a_free;
  uint64_t bar_b_full[2], bar_b_free[2];
  uint64_t bar_acc_full[2], bar_acc_free[2];
  uint32_t tmem_base;
  int abort_flag;
  int n_pe;
  float2 row_state[kBlock];  // (running maximum, running sum) of the rows' odd tiles, handed to the even tiles' threads
  // per epilogue warp: 32 rows x 32 columns of a tile on their way to global memory; the 16-byte chunk q of row r
  // sits at chunk position q ^ (r % 8)
  alignas(16) float stage[8][32 * 32];
};

// Item `idx` of CTA `cta`: positions of the size-sorted order (long strips first) are dealt out in rounds of
// gridDim.x, alternating direction, so every CTA gets a similar number of tiles.
__device__ __forceinline__ bool logits_item(int round, int cta, int n_cta, int n_items, int n_pe, int nt, int* h_slot,
                                            int* mt) {
  const int i = (round & 1) ? (n_cta - 1 - cta) : cta;
  const int pos = round * n_cta + i;
  if (pos >= n_items) return false;
  *mt = nt - 1 - pos / n_pe;
  *h_slot = pos % n_pe;
  return true;
}

__global__ void __launch_bounds__(320, 1)
pe_logits_kernel(const __grid_constant__ LogitsMaps maps, const Dims d, const int32_t* __restrict__ pattern,
                 const SelectPtrs w, int* status) {
  pdl_enter();
  extern __shared__ uint8_t smem_raw[];
  LogitsSmem& s = *reinterpret_cast<LogitsSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    s.abort_flag = 0;
    s.n_pe = w.pe_list[d.hq];
    mbar_init(&s.bar_a_full, 1);
    mbar_init(&s.bar_a_free, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&s.bar_b_full[i], 1);
      mbar_init(&s.bar_b_free[i], 1);
      mbar_init(&s.bar_acc_full[i], 1);
      mbar_init(&s.bar_acc_free[i], 4);  // one arrival per warp of the group that drains the buffer
    }
    fence_mbar_init();
  }
  __syncthreads();
  const int n_pe = s.n_pe;
  if (n_pe == 0) return;  // nothing routed to pooled estimation (uniform over the CTA)
  if (warp == 8) {
    tmem_alloc(&s.tmem_base, 256);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tm = s.tmem_base;
  const int nt = (d.nb + kBlock - 1) / kBlock;
  const int n_items = nt * n_pe, n_cta = gridDim.x, cta = blockIdx.x;

  if (warp == 9) {
    if (lane == 0) {
      // ---- TMA producer: the strip's operands once per item, the K-side operands half by half.  It runs in a
      // thread of its own so that a slot is refilled the moment the MMAs that read it have completed, while the
      // issuing thread sits in the tensor pipe's queue.
      for (int pl = 0; pl < 3; ++pl) {
        prefetch_tmap(&maps.q[pl]);
        prefetch_tmap(&maps.k[pl]);
      }
      bool ok = true;
      uint32_t T = 0;  // tiles loaded so far by this CTA
      for (int round = 0; ok; ++round) {
        int hs, mt;
        if (!logits_item(round, cta, n_cta, n_items, n_pe, nt, &hs, &mt)) break;
        const int h = w.pe_list[hs], kvh = h / d.group;
        // the strip's operands may be replaced once every MMA of the previous item has read them
        if (round > 0) ok = mbar_wait(&s.bar_a_free, (round - 1) & 1, &s.abort_flag);
        if (!ok) break;
        mbar_arrive_expect_tx(&s.bar_a_full, 6u * 16384u);
        for (int pl = 0; pl < 3; ++pl)
          for (int hf = 0; hf < 2; ++hf) tma_load_3d(s.a[pl][hf], &maps.q[pl], &s.bar_a_full, hf * 64, h, mt * kBlock);
        for (int jt = 0; jt <= mt && ok; ++jt, ++T) {
          for (int hf = 0; hf < 2 && ok; ++hf) {
            // slot hf is free once the previous tile's MMAs on it have completed
            if (T > 0) ok = mbar_wait(&s.bar_b_free[hf], (T - 1) & 1, &s.abort_flag);
            if (!ok) break;
            mbar_arrive_expect_tx(&s.bar_b_full[hf], 3u * 16384u);
            for (int pl = 0; pl < 3; ++pl)
              tma_load_3d(s.b[hf][pl], &maps.k[pl], &s.bar_b_full[hf], hf * 64, kvh, jt * kBlock);
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 8) {
    if (lane == 0) {
      // ---- MMA issuer
      constexpr uint32_t idesc = umma_idesc_bf16(128, 128, false, false);
      // (term of Q, term of K), smallest products first
      const int pa[6] = {2, 0, 1, 1, 0, 0}, pb[6] = {0, 2, 1, 0, 1, 0};
      const uint64_t a_desc0 = umma_desc_sw128(smem_u32(s.a[0][0]), 0, 1024);
      const uint64_t b_desc0 = umma_desc_sw128(smem_u32(s.b[0][0]), 0, 1024);
      bool ok = true;
      uint32_t T = 0;               // tiles issued so far by this CTA
      uint32_t acc_uses[2] = {0, 0};  // tiles that went into each accumulator
      for (int round = 0; ok; ++round) {
        int hs, mt;
        if (!logits_item(round, cta, n_cta, n_items, n_pe, nt, &hs, &mt)) break;
        ok = mbar_wait(&s.bar_a_full, round & 1, &s.abort_flag);
        for (int jt = 0; jt <= mt && ok; ++jt, ++T) {
          // even tiles of an item accumulate in buffer 0 (drained by epilogue group 0), odd ones in buffer 1
          const int acc = jt & 1;
          if (acc_uses[acc] > 0) ok = mbar_wait(&s.bar_acc_free[acc], (acc_uses[acc] - 1) & 1, &s.abort_flag);
          ++acc_uses[acc];
          for (int hf = 0; hf < 2 && ok; ++hf) {
            ok = mbar_wait(&s.bar_b_full[hf], T & 1, &s.abort_flag);
            if (!ok) break;
            tc_fence_after_sync();
#pragma unroll
            for (int t = 0; t < 6; ++t)
#pragma unroll
              for (int k4 = 0; k4 < 4; ++k4) {
                // term: 32 KB apart (A) / 16 KB apart (B); 64-dim half: 16 KB (A) / 48 KB (B); 32 B per K step
                const uint64_t ad = a_desc0 + static_cast<uint64_t>((pa[t] * 32768 + hf * 16384 + k4 * 32) >> 4);
                const uint64_t bd = b_desc0 + static_cast<uint64_t>((hf * 49152 + pb[t] * 16384 + k4 * 32) >> 4);
                umma_ss(tm + acc * 128, ad, bd, idesc, (hf > 0 || t > 0 || k4 > 0) ? 1u : 0u);
              }
            umma_commit(&s.bar_b_free[hf]);
            if (hf == 1) {
              umma_commit(&s.bar_acc_full[acc]);
              if (jt == mt) umma_commit(&s.bar_a_free);
            }
          }
        }
      }
    }
    __syncwarp();
  } else {
    // ---- epilogue: one thread per row of the strip and group; group gr drains accumulator gr
    const int gr = warp >> 2, r_ = tid & 127;
    const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const bool vec_ok = (d.nb & 3) == 0;
    bool ok = true;
    uint32_t uses = 0;  // tiles this group has drained
    for (int round = 0; ok; ++round) {
      int hs, mt;
      if (!logits_item(round, cta, n_cta, n_items, n_pe, nt, &hs, &mt)) break;
      const int h = w.pe_list[hs];
      const int m = mt * kBlock + r_;
      const bool row_ok = m < d.nb;
      float M = -INFINITY, S = 0.f;
      for (int jt = gr; jt <= mt && ok; jt += 2, ++uses) {
        ok = mbar_wait_warp(&s.bar_acc_full[gr], uses & 1, &s.abort_flag);
        if (!ok) break;
        tc_fence_after_sync();
        uint32_t r[4][32];
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld_x32(tm + lane_addr + gr * 128 + c * 32, r[c]);
        tmem_ld_wait();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&s.bar_acc_free[gr]);
        const int J0 = jt * kBlock;
        // Tiles left of the strip's diagonal tile are causal in full for every row of the strip; only the
        // diagonal tile (jt == mt) needs per-row column counts.
        const bool full = jt < mt && vec_ok;
        const int n_valid = full ? kBlock : min(kBlock, m - J0 + 1);  // columns J <= m of this tile
        float tmax = -INFINITY;
        if (full) {
          float t0 = -INFINITY, t1 = -INFINITY, t2 = -INFINITY, t3 = -INFINITY;
#pragma unroll
          for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              const float z0 = __uint_as_float(r[c][i]) * d.scale_log2, z1 = __uint_as_float(r[c][i + 1]) * d.scale_log2;
              const float z2 = __uint_as_float(r[c][i + 2]) * d.scale_log2, z3 = __uint_as_float(r[c][i + 3]) * d.scale_log2;
              r[c][i] = __float_as_uint(z0); r[c][i + 1] = __float_as_uint(z1);
              r[c][i + 2] = __float_as_uint(z2); r[c][i + 3] = __float_as_uint(z3);
              t0 = fmaxf(t0, z0); t1 = fmaxf(t1, z1); t2 = fmaxf(t2, z2); t3 = fmaxf(t3, z3);
            }
          tmax = fmaxf(fmaxf(t0, t1), fmaxf(t2, t3));
        } else {
#pragma unroll
          for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const float z = __uint_as_float(r[c][i]) * d.scale_log2;
              r[c][i] = __float_as_uint(z);
              if (c * 32 + i < n_valid) tmax = fmaxf(tmax, z);
            }
        }
        if (row_ok) {
          // (the order of the additions is the same in both branches: the sums must not depend on the path)
          float tsum = 0.f;
          if (full) {
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
              for (int i = 0; i < 32; ++i) tsum += ex2(__uint_as_float(r[c][i]) - tmax);
          } else {
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (c * 32 + i < n_valid) tsum += ex2(__uint_as_float(r[c][i]) - tmax);
          }
          const float nm = fmaxf(M, tmax);
          S = S * ex2(M - nm) + tsum * ex2(tmax - nm);
          M = nm;
        }
        // The thread holds 128 columns of ONE row; stored from here, a warp's store would touch 32 rows (32 lines
        // of 16 bytes each).  The warp passes 32 x 32 chunks through shared memory instead, so that every store
        // writes four rows of 128 contiguous bytes.
        float* stg = s.stage[warp];
        const int m_warp = mt * kBlock + (warp & 3) * 32;  // first row of this warp
        const int rr0 = lane >> 3, qq = lane & 7;          // this lane stores chunk qq of rows rr0, rr0 + 4, ...
        float* dst0 = w.amat + (static_cast<size_t>(h) * d.nb + m_warp + rr0) * d.nb + J0 + 4 * qq;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4)
            *reinterpret_cast<uint4*>(stg + lane * 32 + ((q4 ^ (lane & 7)) << 2)) =
                make_uint4(r[c][4 * q4], r[c][4 * q4 + 1], r[c][4 * q4 + 2], r[c][4 * q4 + 3]);
          __syncwarp();
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const int rr = 4 * kk + rr0;
            const float4 vv = *reinterpret_cast<const float4*>(stg + rr * 32 + ((qq ^ (rr & 7)) << 2));
            const int m_rr = m_warp + rr;
            float* dst = dst0 + static_cast<size_t>(4 * kk) * d.nb + c * 32;
            if (full) {
              if (m_rr < d.nb) *reinterpret_cast<float4*>(dst) = vv;
            } else {
              const int cnt = min(kBlock, m_rr - J0 + 1) - (c * 32 + 4 * qq);  // how many of the four columns are causal
              if (m_rr < d.nb && cnt > 0) {
                if (vec_ok && cnt >= 4) {
                  *reinterpret_cast<float4*>(dst) = vv;
                } else {
                  dst[0] = vv.x;
                  if (cnt > 1) dst[1] = vv.y;
                  if (cnt > 2) dst[2] = vv.z;
                  if (cnt > 3) dst[3] = vv.w;
                }
              }
            }
          }
          __syncwarp();
        }
      }
      // the odd tiles' statistics join the even tiles' (every row has an even tile: tile 0)
      if (gr == 1) s.row_state[r_] = make_float2(M, S);
      named_bar_sync(1, 256);
      if (gr == 0 && ok && row_ok) {
        const float2 o = s.row_state[r_];
        const float nm = fmaxf(M, o.x);
        S = S * ex2(M - nm) + (o.y > 0.f ? o.y * ex2(o.x - nm) : 0.f);
        w.row_m[static_cast<size_t>(h) * d.nb + m] = nm;
        w.row_inv[static_cast<size_t>(h) * d.nb + m] = 1.0f / (S * static_cast<float>(d.nb));
      }
      named_bar_sync(1, 256);  // row_state may be overwritten by the next item
      // a wait that gave up in either group ends both (the flag was set before that group reached the barriers)
      ok = ok && *reinterpret_cast<volatile int*>(&s.abort_flag) == 0;
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (tid == 0 && s.abort_flag) atomicExch(status, CRISP_ERR_DEVICE_TIMEOUT);
  if (warp == 8) tmem_dealloc(tm, 256);
}

// Entry (m, J) of the pooled map: causal row softmax divided by the total N_b.  Every pass computes it with
// these two instructions, so all of them see the same bits.
__device__ __forceinline__ float pe_value(float z, float row_max, float row_inv) { return ex2(z - row_max) * row_inv; }

// ------------------------------------------------------------------------------------------------
// PE heads: gamma cut by radix histogram over the value bits
// ------------------------------------------------------------------------------------------------
// The bin of the current level that holds the cut: the bins are read once, in parallel (largest values first),
// an exclusive block scan gives the mass above every bin, and the first non-empty bin at which the mass reaches
// gamma is the one.  Called by all kHistThreads threads of the last CTA of a head to finish the level.
__device__ void locate_cut(const Dims& d, const SelectPtrs& w, int h, int level, unsigned long long* warp_tot /*[17]*/,
                           int* first_hit) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int kPer = kMaxBins / kHistThreads;  // bins per thread
  const int nbins = level_bins(level);
  const int off = level_offset(level);
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
  // position p (0 = largest values) is bin nbins - 1 - p; thread t owns positions kPer t .. kPer t + kPer - 1.
  // The histograms were built with atomics by other CTAs: read them from L2.
  unsigned long long mm[kPer];
  unsigned int cc[kPer];
  unsigned long long mine = 0ull;
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const int p = kPer * tid + i;
    mm[i] = p < nbins ? __ldcg(gm + (nbins - 1 - p)) : 0ull;
    cc[i] = p < nbins ? __ldcg(gc + (nbins - 1 - p)) : 0u;
    mine += mm[i];
  }
  if (tid == 0) *first_hit = 0x7fffffff;
  unsigned long long incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const unsigned long long wt = lane < kHistThreads / 32 ? warp_tot[lane] : 0ull;
    unsigned long long wi = wt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long t = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += t;
    }
    if (lane < kHistThreads / 32) warp_tot[lane] = wi - wt;  // mass of the warps before this one
    if (lane == 31) warp_tot[16] = wi;                       // total
  }
  __syncthreads();
  unsigned long long before = c.mass_above + warp_tot[warp] + (incl - mine);  // mass above this thread's first position
  int my_hit = 0x7fffffff;
  unsigned long long hit_above = 0ull;
  unsigned int hit_count = 0u;
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    // (a bin is non-empty if it has a count or a mass: only the last level keeps counts on every path)
    if (my_hit == 0x7fffffff && (cc[i] != 0u || mm[i] != 0ull) && before + mm[i] >= gamma) {
      my_hit = kPer * tid + i;
      hit_above = before;
      hit_count = cc[i];
    }
    before += mm[i];
  }
  if (my_hit != 0x7fffffff) atomicMin(first_hit, my_hit);
  __syncthreads();
  const int fp = *first_hit;
  if (fp == 0x7fffffff) {
    if (tid == 0) {
      // the target exceeds the total mass (gamma >= 1 or rounding): keep every causal entry
      c.cutkey = 0u;
      c.take = -1;
      c.mass_above += warp_tot[16];
      w.cut[h] = c;
    }
    return;
  }
  if (fp != my_hit) return;
  // the thread that owns the bin of the cut finishes the level
  const int found = nbins - 1 - fp;
  c.mass_above = hit_above;
  c.prefix |= static_cast<unsigned int>(found) << level_shift(level);
  if (level == 2) {
    c.cutkey = c.prefix;
    // all entries of this bin are equal; t = the smallest count whose mass reaches gamma
    const unsigned long long v = __float2ull_rn(__uint_as_float(c.cutkey) * kMassScale);
    long long t = 1;
    if (v > 0ull) {
      const unsigned long long need = gamma - hit_above;  // > 0 here
      t = static_cast<long long>((need + v - 1ull) / v);
    }
    if (t < 1) t = 1;
    if (t > static_cast<long long>(hit_count)) t = static_cast<long long>(hit_count);
    c.take = t;
  }
  w.cut[h] = c;
}

// Mass bookkeeping of the histograms.  The mass of an entry is its value in 2^-60 fixed point,
// round(v * 2^60); for a value with biased exponent e >= 90 that is exactly its 24-bit significand shifted left
// by e - 90.  All entries of one bin share their exponent at every level (level 0 bins ARE exponents, the
// lower levels only see entries inside the cut's exponent), so a bin's mass is the sum of its entries'
// significands, shifted once when the bin is flushed.  The sum is kept in shared memory as two 32-bit words
// (low and high twelve bits of the significands) next to the count: plain 32-bit adds, no 64-bit atomics.
// A CTA sees fewer than 2^19 entries of a head (host-side grid choice), so none of the words can overflow.
// The rare values below 2^-37 (exponent < 90, zero included) go straight to the global histogram.
constexpr int kMinFastExp = 90;

__device__ __forceinline__ void hist_slow_add(const SelectPtrs& w, int h, int level, int bin, float v) {
  atomicAdd(w.hcount + static_cast<size_t>(h) * kHistStride + level_offset(level) + bin, 1u);
  atomicAdd(w.hmass + static_cast<size_t>(h) * kHistStride + level_offset(level) + bin, __float2ull_rn(v * kMassScale));
}

// One group of 128 consecutive entries of a row (four per lane) at one level.
template <int kLevel, bool kMasked>
__device__ __forceinline__ void hist_group(const float (&z)[4], int J, int m, float M, float inv, unsigned int prefix,
                                           unsigned int* cnt, unsigned int* slo, unsigned int* shi, const SelectPtrs& w,
                                           int h, int lane, int& gt, int& in) {
  unsigned int key[4];
  bool ins[4];
  bool any = false;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    key[e] = __float_as_uint(pe_value(z[e], M, inv));
    const bool valid = !kMasked || J + e <= m;
    if (kLevel == 0) {
      ins[e] = valid;
    } else if (kLevel == 1) {
      ins[e] = valid && (key[e] >> kL0Shift) == (prefix >> kL0Shift);
    } else {
      ins[e] = valid && (key[e] >> kL1Shift) == (prefix >> kL1Shift);
      gt += (valid && (key[e] >> kL1Shift) > (prefix >> kL1Shift)) ? 1 : 0;
      in += ins[e] ? 1 : 0;
    }
    any = any || ins[e];
  }
  if (kLevel > 0 && !__any_sync(0xffffffffu, any)) return;  // nothing of this group lies in the cut's bin
  int bin[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const int b = kLevel == 0 ? static_cast<int>(key[e] >> kL0Shift)
                              : (kLevel == 1 ? static_cast<int>((key[e] >> kL1Shift) & (kL1Bins - 1))
                                             : static_cast<int>(key[e] & (kL2Bins - 1)));
    bin[e] = ins[e] ? b : -1;
    if (ins[e] && (key[e] >> 23) < kMinFastExp) {
      hist_slow_add(w, h, kLevel, b, __uint_as_float(key[e]));
      bin[e] = -1;
    }
  }
  // warp-wide rounds: the bin of the first lane that still holds an entry collects all of its entries in the warp
  constexpr int kRounds = kLevel == 0 ? 3 : 1;
#pragma unroll 1
  for (int round = 0; round < kRounds; ++round) {
    const bool left = (bin[0] & bin[1] & bin[2] & bin[3]) >= 0;  // some bin is not -1
    const uint32_t have = __ballot_sync(0xffffffffu, left);
    if (have == 0u) return;
    const int first = bin[0] >= 0 ? bin[0] : (bin[1] >= 0 ? bin[1] : (bin[2] >= 0 ? bin[2] : bin[3]));
    const int ref = __shfl_sync(0xffffffffu, first, __ffs(have) - 1);
    unsigned int n = 0u, lo = 0u, hi = 0u;
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (bin[e] == ref) {
        ++n;
        lo += key[e] & 0xFFFu;
        hi += ((key[e] >> 12) & 0x7FFu) | 0x800u;
        bin[e] = -1;
      }
    // (counts matter at the last level only: above it a bin that received an entry has a non-zero mass)
    if (kLevel == 2) n = __reduce_add_sync(0xffffffffu, n);
    lo = __reduce_add_sync(0xffffffffu, lo);
    hi = __reduce_add_sync(0xffffffffu, hi);
    if (lane == 0) {
      if (kLevel == 2) atomicAdd(&cnt[ref], n);
      atomicAdd(&slo[ref], lo);
      atomicAdd(&shi[ref], hi);
    }
  }
  // whatever is left goes in lane by lane
#pragma unroll
  for (int e = 0; e < 4; ++e)
    if (bin[e] >= 0) {
      if (kLevel == 2) atomicAdd(&cnt[bin[e]], 1u);
      atomicAdd(&slo[bin[e]], key[e] & 0xFFFu);
      atomicAdd(&shi[bin[e]], ((key[e] >> 12) & 0x7FFu) | 0x800u);
    }
}

// Level 1 of one group of 128 consecutive entries, four per lane.  Every entry the level sees has the cut's
// exponent, and its bin is the upper twelve bits of its mantissa, so a bin's sum of significands is its count
// times a constant plus the sum of the entries' lower eleven bits: count (bits 21-31) and sum (bits 0-20) share
// one 32-bit word `pk` and an entry costs ONE shared-memory add.  The fields hold 1024 entries; the add returns
// the word's old value, and a thread that finds 256 or more entries in it moves the word's content to the
// bin's wide counters (cnt, slo) before its next add, so with 512 threads, each with at most one add between two
// checks, a word never holds more than 256 + 512 entries.  Entries that share the bin of the warp's first pending
// entry are summed across the warp first and go to the wide counters directly (a flat map puts every entry there).
constexpr unsigned int kPkShift = 21, kPkDrain = 256;
template <bool kMasked>
__device__ __forceinline__ void hist1_group(const float (&z)[4], int J, int m, float M, float inv, unsigned int prefix,
                                            unsigned int* cnt, unsigned int* slo, unsigned int* pk, const SelectPtrs& w,
                                            int h, int lane) {
  unsigned int key[4];
  int bin[4];
  bool any = false;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    key[e] = __float_as_uint(pe_value(z[e], M, inv));
    const bool ins = (!kMasked || J + e <= m) && (key[e] >> kL0Shift) == (prefix >> kL0Shift);
    bin[e] = ins ? static_cast<int>((key[e] >> kL1Shift) & (kL1Bins - 1)) : -1;
    any = any || ins;
  }
  if (!__any_sync(0xffffffffu, any)) return;  // nothing of this group lies in the cut's bin
  if ((prefix >> 23) < kMinFastExp) {          // values below 2^-37: straight to the global histogram
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (bin[e] >= 0) hist_slow_add(w, h, 1, bin[e], __uint_as_float(key[e]));
    return;
  }
  {
    const bool left = (bin[0] & bin[1] & bin[2] & bin[3]) >= 0;  // some bin is not -1
    const uint32_t have = __ballot_sync(0xffffffffu, left);
    const int first = bin[0] >= 0 ? bin[0] : (bin[1] >= 0 ? bin[1] : (bin[2] >= 0 ? bin[2] : bin[3]));
    const int ref = __shfl_sync(0xffffffffu, first, __ffs(have) - 1);
    unsigned int n = 0u, lo = 0u;
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (bin[e] == ref && bin[e] >= 0) ++n;
    // worth a warp-wide sum only when the bin is crowded
    if (__reduce_add_sync(0xffffffffu, n) > 8u) {
      n = 0u;
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (bin[e] == ref) {
          ++n;
          lo += key[e] & 0x7FFu;
          bin[e] = -1;
        }
      n = __reduce_add_sync(0xffffffffu, n);
      lo = __reduce_add_sync(0xffffffffu, lo);
      if (lane == 0) {
        atomicAdd(&cnt[ref], n);
        atomicAdd(&slo[ref], lo);
      }
    }
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    if (bin[e] >= 0) {
      const unsigned int old = atomicAdd(&pk[bin[e]], (1u << kPkShift) | (key[e] & 0x7FFu));
      if ((old >> kPkShift) >= kPkDrain) {
        const unsigned int t = atomicExch(&pk[bin[e]], 0u);
        atomicAdd(&cnt[bin[e]], t >> kPkShift);
        atomicAdd(&slo[bin[e]], t & ((1u << kPkShift) - 1u));
      }
    }
    asm volatile("" ::: "memory");  // one add per thread between two checks
  }
}

// Level 0 (bins = exponents) of one group of 128 consecutive entries, four per lane.  An entry is at most the
// row's largest value, 1 / (row sum N_b), so its exponent is e_top - k with k >= 0, and most entries have k < 4.
// Each lane keeps one packed 64-bit accumulator per k in registers - the sum of the 24-bit significands in the
// low word, the count in the high word - and the warp adds them up once per flush
// (hist0_flush), so such an entry costs a handful of integer instructions and no shared-memory traffic.  A group
// in which any lane holds another kind of entry (k >= 4, or a value below 2^-37) takes the general path.
template <bool kMasked>
__device__ __forceinline__ void hist0_group(const float (&z)[4], int J, int m, float M, float inv, int e_top,
                                            unsigned long long (&acc)[4], unsigned int* cnt, unsigned int* slo,
                                            unsigned int* shi, const SelectPtrs& w, int h, int lane) {
  unsigned int key[4];
  bool fast = true;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    key[e] = __float_as_uint(pe_value(z[e], M, inv));
    const bool valid = !kMasked || J + e <= m;
    const int ex = static_cast<int>(key[e] >> 23);
    fast = fast && (!valid || (e_top - ex < 4 && ex >= kMinFastExp));
  }
  if (!__all_sync(0xffffffffu, fast)) {
    int gt = 0, in = 0;
    hist_group<0, kMasked>(z, J, m, M, inv, 0u, cnt, slo, shi, w, h, lane, gt, in);
    return;
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const bool valid = !kMasked || J + e <= m;
    const int k = e_top - static_cast<int>(key[e] >> 23);
    // whole 24-bit significand in the low word (255 entries fit in 32 bits), count in the high word
    const unsigned long long packed = static_cast<unsigned long long>((key[e] & 0x7FFFFFu) | 0x800000u) | (1ull << 32);
#pragma unroll
    for (int b = 0; b < 4; ++b)
      if (valid && k == b) acc[b] += packed;
  }
}
// Adds the lanes' accumulators into the CTA's shared-memory bins e_top .. e_top - 3 and clears them.  A lane may
// hold at most 255 entries per accumulator between two flushes (255 significands fit in 32 bits).
__device__ __forceinline__ void hist0_flush(unsigned long long (&acc)[4], int e_top, unsigned int* cnt,
                                            unsigned int* slo, unsigned int* shi, int lane) {
#pragma unroll
  for (int b = 0; b < 4; ++b) {
    const unsigned int n = static_cast<unsigned int>(acc[b] >> 32);
    if (__any_sync(0xffffffffu, n != 0u)) {
      // the lanes' significand sums in two halves: the low twelve bits and the rest (below 2^20 per lane)
      const unsigned int ns = __reduce_add_sync(0xffffffffu, n);
      const unsigned int lo = __reduce_add_sync(0xffffffffu, static_cast<unsigned int>(acc[b]) & 0xFFFu);
      const unsigned int hi = __reduce_add_sync(0xffffffffu, static_cast<unsigned int>(acc[b]) >> 12);
      if (lane == 0) {
        atomicAdd(&cnt[e_top - b], ns);
        atomicAdd(&slo[e_top - b], lo);
        atomicAdd(&shi[e_top - b], hi);
      }
    }
    acc[b] = 0ull;
  }
}

// Four consecutive logits of a row.  With kVec the row's storage is read as one float4 (columns beyond m but
// inside the row's N_b slots hold unspecified values, which the callers mask); otherwise element by element.
template <bool kVec>
__device__ __forceinline__ void load_z4(const float* __restrict__ row, int J, int m, float (&z)[4]) {
  if (kVec) {
    const float4 v = *reinterpret_cast<const float4*>(row + J);
    z[0] = v.x; z[1] = v.y; z[2] = v.z; z[3] = v.w;
  } else {
#pragma unroll
    for (int e = 0; e < 4; ++e) z[e] = (J + e <= m) ? row[J + e] : 0.f;
  }
}

// One histogram level of one head per CTA column (blockIdx.y = head).  A warp takes one row at a time (rows dealt
// round robin from the longest down), reads its logits as float4 - 512 entries in flight per warp - recomputes
// the normalised values and bins the ones whose upper bits match the prefix found so far.  At level 0 the lanes
// keep the bins of the row's top four exponents in registers (hist0_group).  Elsewhere entries that share a
// bin with the first pending entry of the warp are added across the warp and cost one set of adds (one such round
// at the lower levels, whose entries are spread over thousands of bins unless the map is flat; three in level 0's
// general path); what is left goes in lane by lane.  Level 2 also
// counts, per row, the entries above and inside the cut's last bin.  The last CTA of a head to finish locates
// the cut in the head's finished histogram.
template <int kLevel, bool kVec>
__global__ void __launch_bounds__(kHistThreads)
pe_hist_kernel(const Dims d, const int32_t* __restrict__ pattern, const SelectPtrs w, int resident_ctas, int min_ctas) {
  pdl_enter();
  const int h = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (pattern[h] != CRISP_PATTERN_PE) return;
  // The grid has room for every head being a PE head; how many there are is known only on the device.  The PE
  // heads share the CTAs that fit on the GPU at once evenly, so that the launch is one full wave rather than
  // one and a bit; the CTAs beyond a head's share leave at once.  (min_ctas keeps a CTA's bin sums in 32 bits.)
  const int n_ctas = min(static_cast<int>(gridDim.x), max(min_ctas, resident_ctas / max(1, w.pe_list[d.hq])));
  if (static_cast<int>(blockIdx.x) >= n_ctas) return;
  extern __shared__ uint8_t hist_raw[];
  constexpr int nbins = level_bins(kLevel);
  unsigned int* cnt = reinterpret_cast<unsigned int*>(hist_raw);  // [nbins] each
  unsigned int* slo = cnt + nbins;
  unsigned int* shi = slo + nbins;  // at level 1: the packed count | sum words of hist1_group
  __shared__ unsigned long long warp_tot[17];
  __shared__ int first_hit;
  __shared__ int is_last;
  const CutState cs = w.cut[h];  // written by the previous level's last CTA (an earlier launch)
  const bool skip = kLevel > 0 && cs.take == -1;  // gamma is out of reach: everything is kept
  if (!skip) {
    for (int i = tid; i < 3 * nbins; i += kHistThreads) cnt[i] = 0u;
    __syncthreads();
    const unsigned int prefix = cs.prefix;
    const float* am = w.amat + static_cast<size_t>(h) * d.nb * d.nb;
    const float* rm = w.row_m + static_cast<size_t>(h) * d.nb;
    const float* ri = w.row_inv + static_cast<size_t>(h) * d.nb;
    const int n_warps = n_ctas * (kHistThreads / 32), gw = blockIdx.x * (kHistThreads / 32) + warp;
    for (int m = d.nb - 1 - gw; m >= 0; m -= n_warps) {
      const float* row = am + static_cast<size_t>(m) * d.nb;
      const float M = rm[m], inv = ri[m];
      int gt = 0, in = 0;
      int J0 = 0;
      // level 0: the row's largest value is inv itself (its exponent bounds every entry's), see hist0_group
      const int e_top = static_cast<int>(__float_as_uint(inv) >> 23);
      unsigned long long acc[4] = {0ull, 0ull, 0ull, 0ull};
      // whole steps of 512 entries: the four loads of a lane are issued before any of them is binned
      for (; J0 + 511 <= m; J0 += 512) {
        float z[4][4];
#pragma unroll
        for (int u = 0; u < 4; ++u) load_z4<kVec>(row, J0 + 128 * u + 4 * lane, m, z[u]);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (kLevel == 0) {
            hist0_group<false>(z[u], J0 + 128 * u + 4 * lane, m, M, inv, e_top, acc, cnt, slo, shi, w, h, lane);
          } else if (kLevel == 1) {
            hist1_group<false>(z[u], J0 + 128 * u + 4 * lane, m, M, inv, prefix, cnt, slo, shi, w, h, lane);
          } else {
            hist_group<kLevel, false>(z[u], J0 + 128 * u + 4 * lane, m, M, inv, prefix, cnt, slo, shi, w, h, lane, gt, in);
          }
        }
        // 16 entries per lane and step: flush well before a 20-bit field can overflow
        if (kLevel == 0 && (J0 & (512 * 8 - 1)) == 512 * 7) hist0_flush(acc, e_top, cnt, slo, shi, lane);
      }
      // the rest of the row, 128 entries at a time
      for (; J0 <= m; J0 += 128) {
        float z[4];
        load_z4<kVec>(row, J0 + 4 * lane, m, z);
        if (kLevel == 0) {
          hist0_group<true>(z, J0 + 4 * lane, m, M, inv, e_top, acc, cnt, slo, shi, w, h, lane);
        } else if (kLevel == 1) {
          hist1_group<true>(z, J0 + 4 * lane, m, M, inv, prefix, cnt, slo, shi, w, h, lane);
        } else {
          hist_group<kLevel, true>(z, J0 + 4 * lane, m, M, inv, prefix, cnt, slo, shi, w, h, lane, gt, in);
        }
      }
      if (kLevel == 0) hist0_flush(acc, e_top, cnt, slo, shi, lane);
      if (kLevel == 2) {
        gt = warp_sum_i(gt);
        in = warp_sum_i(in);
        if (lane == 0) {
          w.n_gt[static_cast<size_t>(h) * d.nb + m] = gt;
          w.n_eq[static_cast<size_t>(h) * d.nb + m] = in;
        }
      }
    }
    __syncthreads();
    unsigned int* gc = w.hcount + static_cast<size_t>(h) * kHistStride + level_offset(kLevel);
    unsigned long long* gm = w.hmass + static_cast<size_t>(h) * kHistStride + level_offset(kLevel);
    for (int i = tid; i < nbins; i += kHistThreads)
      if (cnt[i] | slo[i] | shi[i]) {
        // the bin's exponent: its own index at level 0, the cut's exponent below
        const int e = kLevel == 0 ? i : static_cast<int>(prefix >> kL0Shift);
        unsigned long long sig = (static_cast<unsigned long long>(shi[i]) << 12) + slo[i];
        unsigned int n = cnt[i];
        if (kLevel == 1) {
          // shi is the packed word of hist1_group: count | sum of the lower eleven mantissa bits
          n += shi[i] >> kPkShift;
          sig = static_cast<unsigned long long>(n) * (0x800000ull | (static_cast<unsigned long long>(i) << kL1Shift)) +
                slo[i] + (shi[i] & ((1u << kPkShift) - 1u));
        }
        atomicAdd(&gc[i], n);
        atomicAdd(&gm[i], sig << (e - kMinFastExp));
      }
  }
  // the last CTA of this head to get here locates the cut in the finished histogram
  __threadfence();
  __syncthreads();
  if (tid == 0) is_last = atomicAdd(&w.hist_done[kLevel * d.hq + h], 1) == n_ctas - 1;
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  locate_cut(d, w, h, kLevel, warp_tot, &first_hit);
}

// The head-wide part of a PE head's row bookkeeping, run by one CTA of 1024 threads once the per-row counts of the
// entries above the cut's key (n_gt) and equal to it (n_eq) are final: the ties taken per row (in row-major order),
// the forced entries, the row lengths and their scan.
__device__ void pe_rows_finish(const Dims& d, const SelectPtrs& w, int h, const CutState& c, long long* scratch) {
  const int tid = threadIdx.x;
  const size_t base = static_cast<size_t>(h) * d.nb;
  const float* am = w.amat + base * d.nb;
  const int seg = (d.nb + 1023) / 1024;
  const int b0 = min(tid * seg, d.nb), b1 = min(b0 + seg, d.nb);
  long long local = 0;
  if (c.take != -1)
    for (int m = b0; m < b1; ++m) local += __ldcg(&w.n_eq[base + m]);
  long long before = block_exclusive_scan_1024(local, scratch, nullptr);
  long long len_local = 0;
  for (int m = b0; m < b1; ++m) {
    int count, take;
    if (c.take == -1) {
      take = 0;
      count = m + 1;  // every causal entry
    } else {
      const int eq = __ldcg(&w.n_eq[base + m]);
      const long long left = c.take - before;
      take = static_cast<int>(left <= 0 ? 0 : (left >= eq ? eq : left));
      before += eq;
      // the forced entries (column 0 and the diagonal): selected already, or to be added
      const float M = w.row_m[base + m], inv = w.row_inv[base + m];
      const float* row = am + static_cast<size_t>(m) * d.nb;
      const unsigned int k0 = __float_as_uint(pe_value(row[0], M, inv)), km = __float_as_uint(pe_value(row[m], M, inv));
      const bool sel0 = k0 > c.cutkey || (k0 == c.cutkey && take >= 1);   // column 0 is the row's first tie
      const bool selm = km > c.cutkey || (km == c.cutkey && take >= eq);  // the diagonal is its last
      count = __ldcg(&w.n_gt[base + m]) + take + (sel0 ? 0 : 1);
      if (m > 0) count += selm ? 0 : 1;
    }
    w.take[base + m] = take;
    w.counts[base + m] = count;
    len_local += count;
  }
  long long total;
  long long run = block_exclusive_scan_1024(len_local, scratch, &total);
  for (int m = b0; m < b1; ++m) {
    w.local_off[base + m] = static_cast<int>(run);
    run += w.counts[base + m];
  }
  if (tid == 0) w.head_total[h] = total;
}

// ------------------------------------------------------------------------------------------------
// PE heads of short prompts (N_b <= kSmallNb, i.e. up to 8064 tokens): pooled logits, row statistics and the
// gamma cut in one CTA
// ------------------------------------------------------------------------------------------------
// With at most 2016 causal entries per head the tensor-core kernel and the three histogram launches are all
// fixed cost (~70 us together at 4096 tokens).  One CTA per PE head does the same work out of shared memory:
// fp32 dot products of the block means, the rows' maxima and sums, a bitonic sort of the values and a prefix sum
// of their masses in sorted order, which gives the cut directly.  It leaves exactly what pe_logits_kernel and the histogram levels
// leave (the logits, the rows' normalisers, the cut state, and per row the number of entries above the cut's key
// and equal to it) and ends with the head-wide step of pe_rows_kernel, so fill_kernel follows unchanged.
constexpr int kSmallNb = 63;  // 2016 entries: the sort network stays at 2048 keys
constexpr int kSmallPitch = 132;  // floats per block mean in shared memory: 16-byte aligned rows, no bank conflicts
struct SmallSmem {
  float q[kSmallNb * kSmallPitch];
  float k[kSmallNb * kSmallPitch];
  float z[kSmallNb * (kSmallNb + 1) / 2];
  unsigned int key[2048];  // the entries' values as bit patterns, sorted in descending order (zero-padded)
  float row_m[kSmallNb], row_inv[kSmallNb];
  long long scratch[33];
  int first, run_start, run_len;
  unsigned long long above;
  CutState cut;
};
__global__ void __launch_bounds__(1024)
pe_small_kernel(const Dims d, const int32_t* __restrict__ pattern, const SelectPtrs w) {
  pdl_enter();
  const int h = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (pattern[h] != CRISP_PATTERN_PE) return;
  extern __shared__ uint8_t small_raw[];
  SmallSmem& s = *reinterpret_cast<SmallSmem*>(small_raw);
  const int nb = d.nb, n_entries = nb * (nb + 1) / 2, kvh = h / d.group;
  // ---- block means of Q (this head) and K (its KV head)
  const float* qb = w.qbar + static_cast<size_t>(h) * nb * kHeadDim;
  const float* kb = w.kbar + static_cast<size_t>(kvh) * nb * kHeadDim;
  for (int i = tid; i < nb * (kHeadDim / 4); i += 1024) {
    const int r = i / (kHeadDim / 4), c4 = i % (kHeadDim / 4);
    *reinterpret_cast<float4*>(&s.q[r * kSmallPitch + 4 * c4]) = reinterpret_cast<const float4*>(qb)[i];
    *reinterpret_cast<float4*>(&s.k[r * kSmallPitch + 4 * c4]) = reinterpret_cast<const float4*>(kb)[i];
  }
  __syncthreads();
  // ---- pooled logits in base-2 units, entry e = (m, J) in row-major order of the causal triangle
  float* am = w.amat + static_cast<size_t>(h) * nb * nb;
  for (int e = tid; e < n_entries; e += 1024) {
    int m = static_cast<int>((sqrtf(8.0f * static_cast<float>(e) + 1.0f) - 1.0f) * 0.5f);
    while (m * (m + 1) / 2 > e) --m;
    while ((m + 1) * (m + 2) / 2 <= e) ++m;
    const int J = e - m * (m + 1) / 2;
    const float4* qv = reinterpret_cast<const float4*>(&s.q[m * kSmallPitch]);
    const float4* kv = reinterpret_cast<const float4*>(&s.k[J * kSmallPitch]);
    float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
#pragma unroll 8
    for (int c = 0; c < kHeadDim / 4; ++c) {
      const float4 a = qv[c], b = kv[c];
      acc0 = fmaf(a.x, b.x, acc0);
      acc1 = fmaf(a.y, b.y, acc1);
      acc2 = fmaf(a.z, b.z, acc2);
      acc3 = fmaf(a.w, b.w, acc3);
    }
    const float z = ((acc0 + acc1) + (acc2 + acc3)) * d.scale_log2;
    s.z[e] = z;
    am[static_cast<size_t>(m) * nb + J] = z;
  }
  __syncthreads();
  // ---- rows: maximum and 1 / (sum N_b), one warp per row
  for (int m = warp; m < nb; m += 32) {
    const float* zr = &s.z[m * (m + 1) / 2];
    float mx = -INFINITY;
    for (int J = lane; J <= m; J += 32) mx = fmaxf(mx, zr[J]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float sum = 0.f;
    for (int J = lane; J <= m; J += 32) sum += ex2(zr[J] - mx);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) {
      const float inv = 1.0f / (sum * static_cast<float>(nb));
      s.row_m[m] = mx;
      s.row_inv[m] = inv;
      w.row_m[static_cast<size_t>(h) * nb + m] = mx;
      w.row_inv[static_cast<size_t>(h) * nb + m] = inv;
    }
  }
  __syncthreads();
  // ---- the entries' keys (bit patterns of the values), padded with zeros to a power of two and sorted in
  // descending order (bitonic network in shared memory)
  int padded = 1024;
  while (padded < n_entries) padded <<= 1;
  for (int e = tid; e < padded; e += 1024) {
    unsigned int key = 0u;
    if (e < n_entries) {
      int m = static_cast<int>((sqrtf(8.0f * static_cast<float>(e) + 1.0f) - 1.0f) * 0.5f);
      while (m * (m + 1) / 2 > e) --m;
      while ((m + 1) * (m + 2) / 2 <= e) ++m;
      key = __float_as_uint(pe_value(s.z[e], s.row_m[m], s.row_inv[m]));
    }
    s.key[e] = key;
  }
  if (tid == 0) {
    s.first = 0x7fffffff;
    s.run_start = 0;
    s.run_len = 0;
    s.above = 0ull;
  }
  __syncthreads();
  for (int size = 2; size <= padded; size <<= 1)
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int t = tid; t < (padded >> 1); t += 1024) {
        const int lo = ((t & ~(stride - 1)) << 1) | (t & (stride - 1)), hi = lo + stride;  // (stride is a power of two)
        const bool descending = (lo & size) == 0;
        const unsigned int a = s.key[lo], b = s.key[hi];
        if ((a < b) == descending) {
          s.key[lo] = b;
          s.key[hi] = a;
        }
      }
      __syncthreads();
    }
  // ---- the cut: the first position of the sorted order at which the running mass reaches gamma
  const double gd = static_cast<double>(d.gamma) * static_cast<double>(kMassScale);
  const unsigned long long gamma = gd >= 1.8e19 ? 0xffffffffffffffffull : static_cast<unsigned long long>(gd);
  const int per = padded >> 10;  // consecutive positions per thread
  unsigned long long mass[2];
  unsigned long long local = 0ull;
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    mass[i] = i < per ? __float2ull_rn(__uint_as_float(s.key[tid * per + i]) * kMassScale) : 0ull;
    local += mass[i];
  }
  long long total_ll;
  unsigned long long before = static_cast<unsigned long long>(
      block_exclusive_scan_1024(static_cast<long long>(local), s.scratch, &total_ll));  // (the total is below 2^61)
  {
    unsigned long long run = before;
#pragma unroll
    for (int i = 0; i < 2; ++i)
      if (i < per) {
        if (run < gamma && run + mass[i] >= gamma) s.first = tid * per + i;  // exactly one position qualifies
        run += mass[i];
      }
  }
  __syncthreads();
  CutState c;
  c.prefix = 0u;
  c.cutkey = 0u;
  c.mass_above = 0ull;
  c.take = -1;  // the target exceeds the total mass (gamma >= 1 or rounding): keep every causal entry
  if (s.first != 0x7fffffff && s.first < n_entries) {
    const unsigned int cutkey = s.key[s.first];
    // the run of entries equal to the cut's key: where it starts (the mass before it is the mass above the cut)
    // and how long it is
    {
      unsigned long long run = before;
      int mine = 0;
#pragma unroll
      for (int i = 0; i < 2; ++i)
        if (i < per) {
          const int pos = tid * per + i;
          if (s.key[pos] == cutkey && pos < n_entries) {
            ++mine;
            if (pos == 0 || s.key[pos - 1] != cutkey) {
              s.run_start = pos;
              s.above = run;
            }
          }
          run += mass[i];
        }
      if (mine) atomicAdd(&s.run_len, mine);
    }
    __syncthreads();
    // all entries at the cut are equal; t = the smallest count whose mass reaches gamma
    const unsigned long long v = __float2ull_rn(__uint_as_float(cutkey) * kMassScale);
    long long t = 1;
    if (v > 0ull) t = static_cast<long long>((gamma - s.above + v - 1ull) / v);
    if (t < 1) t = 1;
    if (t > s.run_len) t = s.run_len;
    c.prefix = cutkey;
    c.cutkey = cutkey;
    c.mass_above = s.above;
    c.take = t;
  }
  if (tid == 0) {
    s.cut = c;
    w.cut[h] = c;
  }
  // ---- per row: entries above the cut's key and equal to it
  if (c.take != -1)
  for (int m = warp; m < nb; m += 32) {
    const float* zr = &s.z[m * (m + 1) / 2];
    const float M = s.row_m[m], inv = s.row_inv[m];
    int gt = 0, eq = 0;
    for (int J = lane; J <= m; J += 32) {
      const unsigned int kk = __float_as_uint(pe_value(zr[J], M, inv));
      gt += kk > c.cutkey;
      eq += kk == c.cutkey;
    }
    gt = warp_sum_i(gt);
    eq = warp_sum_i(eq);
    if (lane == 0) {
      w.n_gt[static_cast<size_t>(h) * nb + m] = gt;
      w.n_eq[static_cast<size_t>(h) * nb + m] = eq;
    }
  }
  // ---- ties per row, row lengths, their scan (what pe_rows_kernel does for the long prompts)
  __syncthreads();
  pe_rows_finish(d, w, h, c, s.scratch);
}

// Per PE head: exact per-row counts of the entries above and tied with the cut, the ties taken per row (in
// row-major order: row m takes clamp(T - ties in rows < m, 0, ties_m)), the row lengths and their prefix sum.
// Only rows with an entry inside the cut's last bin (2048 adjacent fp32 values) are read again; the last CTA of a head to finish
// does the head-wide part.
__global__ void __launch_bounds__(1024)
pe_rows_kernel(const Dims d, const int32_t* __restrict__ pattern, const SelectPtrs w) {
  pdl_enter();
  const int h = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (pattern[h] != CRISP_PATTERN_PE) return;
  __shared__ long long scratch[33];
  __shared__ int is_last;
  const CutState c = w.cut[h];
  const size_t base = static_cast<size_t>(h) * d.nb;
  const float* am = w.amat + base * d.nb;
  if (c.take != -1) {
    const int n_warps = gridDim.x * 32, gw = blockIdx.x * 32 + warp;
    for (int m = gw; m < d.nb; m += n_warps) {
      if (w.n_eq[base + m] == 0) continue;  // no entry inside the cut's bin: the counts of level 2 are exact
      const float* row = am + static_cast<size_t>(m) * d.nb;
      const float M = w.row_m[base + m], inv = w.row_inv[base + m];
      int gt = 0, eq = 0;
      for (int J = lane; J <= m; J += 32) {
        const unsigned int key = __float_as_uint(pe_value(row[J], M, inv));
        gt += key > c.cutkey;
        eq += key == c.cutkey;
      }
      gt = warp_sum_i(gt);
      eq = warp_sum_i(eq);
      if (lane == 0) {
        w.n_gt[base + m] = gt;
        w.n_eq[base + m] = eq;
      }
    }
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) is_last = atomicAdd(&w.rows_done[h], 1) == static_cast<int>(gridDim.x) - 1;
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  pe_rows_finish(d, w, h, c, scratch);
}

// ------------------------------------------------------------------------------------------------
// Global offsets and the lists
// ------------------------------------------------------------------------------------------------
// The kept columns of one PE row, in ascending order, straight to the list.  A warp takes the row 32 consecutive
// entries at a time (lane l holds column J0 + 32 u + l), so the kept entries of a group are the set bits of one
// ballot, their places in the list the bit counts below each lane, and the group leaves as one store to
// consecutive addresses - no scan, no staging.  Sixteen groups' loads are in flight per lane.
template <bool kEdge>
__device__ __forceinline__ void fill_step(const float* __restrict__ row, int J0, int m, float M, float inv,
                                          unsigned int cutkey, bool all, int take, int& ties_seen, int& written,
                                          int32_t* __restrict__ out, int lane) {
  constexpr int kGroups = 16;
  const unsigned int below = (1u << lane) - 1u;
  float z[kGroups];
#pragma unroll
  for (int u = 0; u < kGroups; ++u) {
    const int J = J0 + 32 * u + lane;
    z[u] = (!kEdge || J <= m) ? __ldcs(row + J) : 0.f;
  }
#pragma unroll
  for (int u = 0; u < kGroups; ++u) {
    const int J = J0 + 32 * u + lane;
    if (kEdge && J0 + 32 * u > m) break;  // warp-uniform
    const bool valid = !kEdge || J <= m;
    const unsigned int key = __float_as_uint(pe_value(z[u], M, inv));
    bool keep = valid && (all || key > cutkey || J == 0 || J == m);
    const bool eq = valid && !all && key == cutkey;
    // ties are rare: the first `take` of a row's ties, in column order, are kept
    const unsigned int eq_bits = __ballot_sync(0xffffffffu, eq);
    if (eq_bits != 0u) {
      if (eq && ties_seen + __popc(eq_bits & below) < take) keep = true;
      ties_seen += __popc(eq_bits);
    }
    const unsigned int keep_bits = __ballot_sync(0xffffffffu, keep);
    if (keep) out[written + __popc(keep_bits & below)] = J;
    written += __popc(keep_bits);
  }
}

__device__ __forceinline__ void fill_pe_row(const float* __restrict__ row, int m, float M, float inv, unsigned int cutkey,
                                            bool all, int take, int32_t* __restrict__ out, int lane) {
  int written = 0, ties_seen = 0;
  for (int J0 = 0; J0 <= m; J0 += 512) {
    if (J0 + 511 < m) {  // the step lies inside the row and does not hold the diagonal
      fill_step<false>(row, J0, m, M, inv, cutkey, all, take, ties_seen, written, out, lane);
    } else {
      fill_step<true>(row, J0, m, M, inv, cutkey, all, take, ties_seen, written, out, lane);
    }
  }
}

__global__ void __launch_bounds__(256)
fill_kernel(const Dims d, const int32_t* __restrict__ pattern, const SelectPtrs w, int64_t* __restrict__ row_ptr,
            int32_t* __restrict__ col_idx, int64_t capacity, int64_t* __restrict__ nnz_needed, int* status) {
  pdl_enter();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // CTAs that start together hold the same rows of different heads, so the cheap rows of the VS heads run under
  // the memory traffic of the PE heads' rows
  const int h = blockIdx.x;
  // offsets of the heads: every CTA adds the (few) head totals itself
  __shared__ long long s_base, s_total;
  __shared__ int stage_all[8][1024];  // VS rows: the entries of 32 bitmap words
  if (threadIdx.x < 32) {
    long long before = 0, all = 0;
    for (int hh = lane; hh < d.hq; hh += 32) {
      const long long t = w.head_total[hh];
      all += t;
      if (hh < h) before += t;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      before += __shfl_xor_sync(0xffffffffu, before, o);
      all += __shfl_xor_sync(0xffffffffu, all, o);
    }
    if (lane == 0) {
      s_base = before;
      s_total = all;
    }
  }
  __syncthreads();
  const long long head_base = s_base, total = s_total;
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
    *nnz_needed = total;
    if (total > capacity) atomicExch(status, CRISP_ERR_CAPACITY);
  }
  // long rows first, so that the tail of the launch is made of short ones
  const int m = d.nb - 1 - (blockIdx.y * 8 + warp);
  if (m < 0) return;
  const size_t rbase = static_cast<size_t>(h) * d.nb;
  const long long start = head_base + w.local_off[rbase + m];
  if (lane == 0) {
    row_ptr[static_cast<size_t>(h) * (d.nb + 1) + m] = start;
    if (m == d.nb - 1) row_ptr[static_cast<size_t>(h) * (d.nb + 1) + d.nb] = head_base + w.head_total[h];
  }
  if (total > capacity) return;  // the lists do not fit: col_idx stays untouched
  int32_t* out = col_idx + start;
  if (pattern[h] == CRISP_PATTERN_VS) {
    int written = 0;
    const uint32_t* selv = w.selv + static_cast<size_t>(h) * w.words;
    const uint32_t* selsr = w.selsr + static_cast<size_t>(h) * (w.words + 2);
    const int nwords = (m >> 5) + 1;
    int* stage = stage_all[warp];
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
      // every lane unpacks its own word into the warp's staging area (a word holds a handful of entries, so this
      // takes as many rounds as the fullest word has bits), then the chunk leaves as contiguous 128-byte stores
      const int n_chunk = __shfl_sync(0xffffffffu, incl, 31);
      int pos = incl - c;
      while (bits != 0u) {
        stage[pos++] = wd * 32 + __ffs(bits) - 1;
        bits &= bits - 1u;
      }
      __syncwarp();
      for (int i = lane; i < n_chunk; i += 32) out[written + i] = stage[i];
      __syncwarp();
      written += n_chunk;
    }
  } else {
    const CutState c = w.cut[h];
    const float* row = w.amat + (rbase + m) * d.nb;
    const float M = w.row_m[rbase + m], inv = w.row_inv[rbase + m];
    const int take = w.take[rbase + m];
    fill_pe_row(row, m, M, inv, c.cutkey, c.take == -1, take, out, lane);
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
  // zeroed region first (directly behind the header, so one memset covers both)
  w.hcount = static_cast<unsigned int*>(take(sizeof(unsigned int) * d.hq * kHistStride));
  w.hmass = static_cast<unsigned long long*>(take(sizeof(unsigned long long) * d.hq * kHistStride));
  w.hist_done = static_cast<int*>(take(sizeof(int) * 3 * d.hq));
  w.rows_done = static_cast<int*>(take(sizeof(int) * d.hq));
  w.zero_bytes = off;
  w.selv = static_cast<uint32_t*>(take(sizeof(uint32_t) * d.hq * w.words));
  w.selsr = static_cast<uint32_t*>(take(sizeof(uint32_t) * d.hq * (w.words + 2)));
  w.kbar = static_cast<float*>(take(sizeof(float) * d.hkv * d.nb * kHeadDim));
  w.qbar = static_cast<float*>(take(sizeof(float) * static_cast<size_t>(d.hq) * d.nb * kHeadDim));
  w.ksplit = static_cast<__nv_bfloat16*>(take(sizeof(__nv_bfloat16) * 3 * static_cast<size_t>(d.hkv) * d.nb * kHeadDim));
  w.qsplit = static_cast<__nv_bfloat16*>(take(sizeof(__nv_bfloat16) * 3 * static_cast<size_t>(d.hq) * d.nb * kHeadDim));
  w.amat = static_cast<float*>(take(sizeof(float) * static_cast<size_t>(d.hq) * d.nb * d.nb));
  w.row_m = static_cast<float*>(take(sizeof(float) * d.hq * d.nb));
  w.row_inv = static_cast<float*>(take(sizeof(float) * d.hq * d.nb));
  w.cut = static_cast<CutState*>(take(sizeof(CutState) * d.hq));
  w.n_gt = static_cast<int*>(take(sizeof(int) * d.hq * d.nb));
  w.n_eq = static_cast<int*>(take(sizeof(int) * d.hq * d.nb));
  w.counts = static_cast<int*>(take(sizeof(int) * d.hq * d.nb));
  w.take = static_cast<int*>(take(sizeof(int) * d.hq * d.nb));
  w.local_off = static_cast<int*>(take(sizeof(int) * d.hq * d.nb));
  w.head_total = static_cast<long long*>(take(sizeof(long long) * d.hq));
  w.pe_list = static_cast<int*>(take(sizeof(int) * (d.hq + 1)));
  *total = off;
  return w;
}

int launch_prepare(const Dims& d, const __nv_bfloat16* qb, const __nv_bfloat16* kb, const int32_t* pattern,
                   const float* p_v, const float* p_s, const SelectPtrs& w, int vs_ctas, int pool_all_k,
                   cudaStream_t stream) {
  const size_t vs_smem = (sizeof(double) + sizeof(float) + sizeof(int) + 1) * static_cast<size_t>(d.nb) + 16;
  CRISP_CUDA_TRY(cudaFuncSetAttribute(prepare_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      static_cast<int>(vs_smem)),
                 "select: smem attribute");
  const long long n_tiles = static_cast<long long>(d.nb) * (d.hkv + d.hq);
  const int pool_ctas = static_cast<int>((n_tiles + 7) / 8);
  CRISP_KERNEL("prepare", stream, launch_pdl(prepare_kernel, dim3(vs_ctas + pool_ctas), dim3(1024), vs_smem, stream, 
                                      d, qb, kb, pattern, p_v, p_s, w, vs_ctas, pool_all_k));
  return CRISP_OK;
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
  if (d.nb > 8192 || d.hq > 1024) return CRISP_ERR_UNSUPPORTED;
  size_t total;
  SelectPtrs w = carve(d, ws, &total);
  int* status = static_cast<int*>(ws);
  // status word, histograms and completion counters
  CRISP_CUDA_TRY(cudaMemsetAsync(ws, 0, w.zero_bytes, stream), "select: clear");

  // VS heads: selection and list lengths; PE heads: block means (the PE kernels return at once for VS heads)
  int rc = launch_prepare(d, static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k), pattern, p_v,
                          p_s, w, d.hq, 0, stream);
  if (rc != CRISP_OK) return rc;
  int dev = 0, n_sm = 0;
  CRISP_CUDA_TRY(cudaGetDevice(&dev), "select: device");
  CRISP_CUDA_TRY(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev), "select: SM count");
  if (d.nb <= kSmallNb) {
    // short prompt: logits, row statistics and the cut of a PE head in one CTA
    CRISP_CUDA_TRY(cudaFuncSetAttribute(pe_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(sizeof(SmallSmem))),
                   "select: smem attribute");
    CRISP_KERNEL("pe_small", stream, launch_pdl(pe_small_kernel, dim3(d.hq), dim3(1024), sizeof(SmallSmem), stream, d, pattern, w));
  } else {
    {
      LogitsMaps maps;
      for (int pl = 0; pl < 3; ++pl) {
        rc = make_tmap_bf16_nhd(&maps.q[pl], w.qsplit + static_cast<size_t>(pl) * d.nb * d.hq * kHeadDim, d.nb, d.hq);
        if (rc != CRISP_OK) return rc;
        rc = make_tmap_bf16_nhd(&maps.k[pl], w.ksplit + static_cast<size_t>(pl) * d.nb * d.hkv * kHeadDim, d.nb, d.hkv);
        if (rc != CRISP_OK) return rc;
      }
      const size_t smem = sizeof(LogitsSmem) + 1024;
      CRISP_CUDA_TRY(cudaFuncSetAttribute(pe_logits_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(smem)),
                     "select: smem attribute");
      const int nt = (d.nb + kBlock - 1) / kBlock;
      const int grid = min(n_sm, nt * d.hq);
      CRISP_KERNEL("pe_logits", stream, launch_pdl(pe_logits_kernel, dim3(grid), dim3(320), smem, stream, maps, d, pattern, w, status));
    }
    // histogram passes: a warp takes a row at a time; the grid is sized for a single PE head, the kernel uses as many
    // CTAs per head as make one full wave over the PE heads there are
    const long long causal = static_cast<long long>(d.nb) * (d.nb + 1) / 2;
    // two CTAs of kHistThreads fit on an SM; a CTA must see fewer than 2^19 entries of a head (its 32-bit bin sums)
    const int resident_ctas = 2 * n_sm;
    const int min_ctas = static_cast<int>((causal + (1 << 19) - 1) >> 19);
    const int hist_ctas = max(min_ctas, max(1, min((d.nb + 15) / 16, 64)));
    auto hist_smem = [](int level) { return static_cast<size_t>(level_bins(level)) * 12; };
    const bool vec = (d.nb & 3) == 0;  // rows start on 16-byte boundaries
    auto* hist0 = vec ? pe_hist_kernel<0, true> : pe_hist_kernel<0, false>;
    auto* hist1 = vec ? pe_hist_kernel<1, true> : pe_hist_kernel<1, false>;
    auto* hist2 = vec ? pe_hist_kernel<2, true> : pe_hist_kernel<2, false>;
    CRISP_CUDA_TRY(cudaFuncSetAttribute(hist1, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(hist_smem(1))),
                   "select: smem attribute");
    CRISP_KERNEL("pe_hist0", stream, launch_pdl(hist0, dim3(hist_ctas, d.hq), dim3(kHistThreads), hist_smem(0), stream, d, pattern, w, resident_ctas, min_ctas));
    CRISP_KERNEL("pe_hist1", stream, launch_pdl(hist1, dim3(hist_ctas, d.hq), dim3(kHistThreads), hist_smem(1), stream, d, pattern, w, resident_ctas, min_ctas));
    CRISP_KERNEL("pe_hist2", stream, launch_pdl(hist2, dim3(hist_ctas, d.hq), dim3(kHistThreads), hist_smem(2), stream, d, pattern, w, resident_ctas, min_ctas));
  }
  if (d.nb > kSmallNb) {  // (pe_small_kernel ends with the same step)
    const int rows_ctas = max(1, min((d.nb + 31) / 32, 8));
    CRISP_KERNEL("pe_rows", stream, launch_pdl(pe_rows_kernel, dim3(rows_ctas, d.hq), dim3(1024), 0, stream, d, pattern, w));
  }
  CRISP_KERNEL("fill", stream, launch_pdl(fill_kernel, dim3(d.hq, (d.nb + 7) / 8), dim3(256), 0, stream, 
                                   d, pattern, w, row_ptr, col_idx, capacity, nnz_needed, status));
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
  pdl_enter();
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
  // block means of K for every KV head (no VS work, no Q pooling)
  int rc = launch_prepare(d, nullptr, static_cast<const __nv_bfloat16*>(k), nullptr, nullptr, nullptr, w, 0, 1, stream);
  if (rc != CRISP_OK) return rc;
  CRISP_KERNEL("jsd", stream, launch_pdl(jsd_kernel, dim3(d.hq), dim3(256), sizeof(float) * d.nb, stream, d, static_cast<const __nv_bfloat16*>(q), w.kbar, p_v,
                                                         tau_jsd, jsd, pattern));
  CRISP_CUDA_TRY(cudaGetLastError(), "route_jsd: launch");
  return CRISP_OK;
}

}  // namespace crisp
