// Stage 4: block-sparse (and dense) causal attention (Eq. 1) on tcgen05 tensor cores.
//
// One CTA processes work items; an item is one query head and a PAIR of adjacent query blocks
// (two 128-row tiles).  Both tiles share every K/V block that TMA brings into shared memory, which
// halves the L2 -> shared-memory traffic per flop.  The key blocks of the pair are the sorted union
// of the two blocks' lists, each with two flags saying which tile uses it; the union is never stored: the
// producer and the issuers form it on the fly by a two-way merge of the two lists (EntryStream), and a tile's
// softmax warps walk that tile's own list (TileReader).  (When the pairs of a problem
// do not even fill the SMs, an item is a single query block instead: tile 1 stays idle, the CTAs are twice as many
// and a block alone steps faster than a pair.)
//
// Warp roles (384 threads):
//   warps 0-3   softmax of tile 0 (one thread per query row; TMEM lanes 0-127)
//   warps 4-7   softmax of tile 1
//   warp  8     TMA producer (one thread): Q once per item, K and V blocks through one five-slot ring
//   warps 9,10  MMA issuers, one thread per tile: S_t = Q_t K^T (SS) and O_t += P_t V (P read from TMEM)
//   warp  11    pulls the lines of an item's lists into L2 when the item starts (sparse kernel; hints only)
// TMEM (512 columns): S_0 | S_1 | O_0 | O_1, 128 fp32 columns each.  Every key block is worked on in two
// halves of 64 keys (A, B): S_A and S_B are separate MMAs (N = 64) into the two halves of S_t, and P_t (bf16)
// is written over the columns of S_B.  The columns of S_A are therefore free as soon as the softmax has read
// both halves, so Q K_A^T of the NEXT step is issued behind P_A V_A, in the middle of the current step, and
// Q K_B^T behind P_B V_B at its end: the softmax of the next step finds its first half waiting and receives
// the second while it works on the first.  Neither the softmax nor the tensor pipe waits for a whole step of
// the other, which a whole-block S (P aliased on it) forces: there the per-tile chain Q K^T -> softmax ->
// P V -> Q K^T is serial and two tiles cover only about half of the pipe's time.  The price is that an N = 64
// MMA with both operands in shared memory is bound by operand fetch (58 cycles instead of 32, measured).
// Each half is one step of the online softmax, which rescales O lazily, only when the running maximum
// grows by more than 2^8, and does it in place in TMEM.
// Both issuers see every load of the K/V ring in order and release every slot once, so the ring never runs
// ahead of either tile; apart from that the two tiles run free of each other, except that tile 0's softmax warps
// trail tile 1's by part of a run of exponentials (see the pacing in the softmax branch).
// Work items are handed out dynamically: the producer takes the next position of the cost-sorted order from
// a device counter and passes it to the other roles through a four-slot queue, which balances the load and
// keeps the CTAs that run at the same time on the same K/V blocks (they share them through L2).
// Measured alternatives that were slower and are not kept: a single issuing thread for both tiles (its scalar
// bookkeeping between bursts, several hundred cycles, is idle pipe time); whole-block steps with one issuer
// per tile, with and without handing P over in two halves; computing part of the exponentials on the FMA
// pipe (see kPolyEvery).
// Every mbarrier wait is bounded; a wait that gives up sets a flag that ends all roles, and the
// status word reports CRISP_ERR_DEVICE_TIMEOUT.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace crisp {
using namespace sm100;

namespace {

constexpr uint32_t kFlag0 = 1u << 30, kFlag1 = 1u << 31, kColMask = kFlag0 - 1u;
constexpr float kRescaleThreshold = 8.0f;  // log2 units
constexpr int kStages = 5;                 // K/V ring slots of 32 KB

struct PrefillArgs {
  const int32_t* col_idx;  // the heads' lists (sparse only)
  const int64_t* row_ptr;  // [hq][nb+1]
  const int* order;        // [n_items] item ids sorted by decreasing cost (sparse only)
  __nv_bfloat16* o;        // [n][hq][128]
  float* lse;              // [hq][n] or null
  int* status;
  int n_pairs;             // items per head
  int rows_per_item;       // 2: an item is a pair of query blocks; 1: a single block (small problems)
  int n_items;
  int group_kv;            // 1: schedule one KV head at a time, 0: one global order by cost (small problems)
  const int* gate;         // optional device word: when non-zero the lists are invalid and nothing is done
  int* next_item;          // device counter (zero at launch): position of the next item nobody has taken yet
};

struct PrefillSmem {
  alignas(1024) uint8_t q[2][2][16384];  // [tile][half]
  alignas(1024) uint8_t kv[kStages][2][16384];  // ring of K and V blocks [slot][half]; load 2e is K_e, 2e+1 is V_e
  uint64_t q_full, q_free;
  uint64_t in_exp[4];  // per scheduler: odd phase while tile 1's warp is in the first part of its exponentials
  uint64_t kv_full[kStages], kv_empty[kStages];
  // per tile and per 64-key half (A = keys 0-63, B = keys 64-127 of the block)
  uint64_t s_full[2][2], p_ready[2][2], o_done[2][2];
  // items are handed out dynamically: the producer takes the next position from a device counter and passes
  // it to the other roles through a four-slot queue
  uint64_t itm_full[4], itm_empty[4];
  int item_q[4];
  uint32_t tmem_base;
  int abort_flag;
};

struct Item {
  int h, kvh, m0, m1;
  bool tile1;
  int n_entries;    // dense: key blocks of the item; sparse: unused (the union's length is found by walking it)
  int n0, n1;       // sparse: lengths of the two query blocks' lists (n1 = 0 without a second tile)
  long long base0;  // sparse: offset of block m0's list in col_idx; block m1's follows it
};

template <bool kDense>
__device__ __forceinline__ Item decode_item(int pos, const Dims& d, const PrefillArgs& a) {
  Item it;
  // Item id = (n_pairs - 1 - u) * H_q + h.  Dense: positions walk one KV head at a time (its G query
  // heads interleaved, long rows first), so the CTAs running at any moment stream the same K/V blocks
  // and share them in L2.  Sparse: the same grouping, sorted by cost inside each KV head.
  int idx;
  if (kDense && !a.group_kv) {
    idx = pos;
  } else if (kDense) {
    const int per_kv = a.n_pairs * d.group;
    const int kvh = pos / per_kv, rem = pos % per_kv;
    idx = (rem / d.group) * d.hq + kvh * d.group + rem % d.group;
  } else {
    idx = a.order[pos];
  }
  it.h = idx % d.hq;
  const int u = a.n_pairs - 1 - idx / d.hq;  // long rows first
  it.kvh = it.h / d.group;
  it.m0 = a.rows_per_item * u;
  it.m1 = it.m0 + 1;
  it.tile1 = a.rows_per_item == 2 && it.m1 < d.nb;
  if (kDense) {
    it.n_entries = it.tile1 ? it.m1 + 1 : it.m0 + 1;
    it.n0 = it.n1 = 0;
    it.base0 = 0;
  } else {
    const int64_t* rp = a.row_ptr + static_cast<size_t>(it.h) * (d.nb + 1) + it.m0;
    it.n_entries = 0;
    it.base0 = rp[0];
    it.n0 = static_cast<int>(rp[1] - rp[0]);
    it.n1 = it.tile1 ? static_cast<int>(rp[2] - rp[1]) : 0;
  }
  return it;
}

// The key blocks of ONE tile of an item, in order (what its softmax warps walk: they need neither the other
// tile's blocks nor the position of a block in the K/V stream).  Sparse lists are fetched 32 entries at a time,
// one per lane, and broadcast with a shuffle; all 32 lanes of the warp must call get together.  The fetch runs
// one group of 32 ahead, so that its latency (the lists of a long prompt come from DRAM) never stalls the
// softmax, which is the critical path of a step.
template <bool kDense>
struct TileReader {
  const int32_t* list;
  uint32_t chunk, chunk_next;
  int n;  // blocks of the tile
  __device__ __forceinline__ void init(const Item& it, const PrefillArgs& a, int t, int lane) {
    if (kDense) {
      list = nullptr;
      n = (t == 0 ? it.m0 : it.m1) + 1;
      chunk = chunk_next = 0;
    } else {
      list = a.col_idx + it.base0 + (t == 0 ? 0 : it.n0);
      n = t == 0 ? it.n0 : it.n1;
      chunk = lane < n ? static_cast<uint32_t>(__ldg(list + lane)) : 0u;
      chunk_next = 32 + lane < n ? static_cast<uint32_t>(__ldg(list + 32 + lane)) : 0u;
    }
  }
  __device__ __forceinline__ int get(int i, int lane) {
    if (kDense) return i;
    if ((i & 31) == 0 && i > 0) {
      chunk = chunk_next;
      chunk_next = (i + 32 + lane < n) ? static_cast<uint32_t>(__ldg(list + i + 32 + lane)) : 0u;
    }
    return static_cast<int>(__shfl_sync(0xffffffffu, chunk, i & 31));
  }
};

// Register budgets after setmaxnreg.  The CTA's pool is what the launch allocated (384 threads x 168
// registers); setmaxnreg.inc waits, without a bound, until the pool can serve it, so the budgets of the
// three warpgroups must never add up to more than the pool.
constexpr int kRegsSoftmax = 192, kRegsOther = 112, kRegsLaunch = 168;
static_assert(256 * kRegsSoftmax + 128 * kRegsOther <= 384 * kRegsLaunch, "setmaxnreg budgets exceed the CTA's pool");

template <int N>
__device__ __forceinline__ void reg_alloc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void reg_dealloc() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}

// ---- packed fp32x2 arithmetic (two lanes per instruction on the FMA pipe)
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t v;
  asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
  return v;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// 2^t for a pair of values on the FMA pipe instead of the MUFU: t = n + f with n = round(t),
// f in [-0.5, 0.5]; 2^f by a degree-4 minimax polynomial (max relative error 2.6e-6, far below the
// bf16 rounding of P); 2^n by adding n to the exponent field.  t is clamped at -125.
__device__ __forceinline__ void exp2_poly2(uint64_t t2, float& p0, float& p1) {
  float t0, t1;
  unpack2(t2, t0, t1);
  t0 = fmaxf(t0, -125.0f);
  t1 = fmaxf(t1, -125.0f);
  t2 = pack2(t0, t1);
  const uint64_t magic = pack2(12582912.0f, 12582912.0f);      // 1.5 * 2^23: rounds to an integer
  const uint64_t neg_magic = pack2(-12582912.0f, -12582912.0f);
  const uint64_t neg_one = pack2(-1.0f, -1.0f);
  const uint64_t r2 = add2(t2, magic);
  const uint64_t n2 = add2(r2, neg_magic);
  const uint64_t f2 = fma2(n2, neg_one, t2);
  uint64_t q2 = fma2(f2, pack2(0.009570101276040077f, 0.009570101276040077f),
                     pack2(0.05591785907745361f, 0.05591785907745361f));
  q2 = fma2(q2, f2, pack2(0.240247443318367f, 0.240247443318367f));
  q2 = fma2(q2, f2, pack2(0.6931217908859253f, 0.6931217908859253f));
  q2 = fma2(q2, f2, pack2(0.9999992847442627f, 0.9999992847442627f));
  float r0, r1, q0, q1;
  unpack2(r2, r0, r1);
  unpack2(q2, q0, q1);
  p0 = __int_as_float(__float_as_int(q0) + (__float_as_int(r0) << 23));
  p1 = __int_as_float(__float_as_int(q1) + (__float_as_int(r1) << 23));
}

// Maximum of 64 raw logits of one row (keys key0 .. key0 + 63 of the block); on the diagonal block only
// keys j <= r are visible.
template <bool kDiag>
__device__ __forceinline__ float row_max(const uint32_t (&x)[2][32], int r, int key0) {
  float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
  for (int c = 0; c < 2; ++c)
#pragma unroll
    for (int i = 0; i < 32; i += 8) {
      float a[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        a[u] = __uint_as_float(x[c][i + u]);
        if (kDiag && (key0 + c * 32 + i + u) > r) a[u] = -INFINITY;
      }
      m0 = max3(m0, a[0], a[1]);
      m1 = max3(m1, a[2], a[3]);
      m2 = max3(m2, a[4], a[5]);
      m3 = max3(m3, a[6], a[7]);
    }
  return fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
}

// P = 2^(x * scale - m) for 64 keys as bf16 pairs (two keys per 32-bit word); returns the fp32 row sum.
// With kPolyEvery > 0 one pair in every kPolyEvery goes through exp2_poly2 (FMA pipe) instead of the MUFU.
#ifndef CRISP_POLY_EVERY
#define CRISP_POLY_EVERY 0
#endif
constexpr int kPolyEvery = CRISP_POLY_EVERY;
// `release` is called once, after kPaceRelease of the 32 pairs (see the pacing of the two tiles in the kernel).
constexpr int kPaceRelease = 12;
template <bool kDiag, class Release>
__device__ __forceinline__ float exp_pack(const uint32_t (&x)[2][32], int r, int key0, float scale_log2, float m_used,
                                          uint32_t (&pk)[2][16], Release release) {
  const uint64_t scale2 = pack2(scale_log2, scale_log2);
  const uint64_t negm2 = pack2(-m_used, -m_used);
  uint64_t sum_a = pack2(0.f, 0.f), sum_b = pack2(0.f, 0.f);
#pragma unroll
  for (int c = 0; c < 2; ++c) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const uint64_t t2 = fma2(pack2(__uint_as_float(x[c][2 * i]), __uint_as_float(x[c][2 * i + 1])), scale2, negm2);
      float p0, p1;
      if (kPolyEvery > 0 && (i % (kPolyEvery > 0 ? kPolyEvery : 1)) == kPolyEvery - 1) {
        exp2_poly2(t2, p0, p1);
      } else {
        float t0, t1;
        unpack2(t2, t0, t1);
        p0 = ex2(t0);
        p1 = ex2(t1);
      }
      if (kDiag) {
        if (key0 + c * 32 + 2 * i > r) p0 = 0.f;
        if (key0 + c * 32 + 2 * i + 1 > r) p1 = 0.f;
      }
      if (i & 1) {
        sum_a = add2(sum_a, pack2(p0, p1));
      } else {
        sum_b = add2(sum_b, pack2(p0, p1));
      }
      pk[c][i] = pack_bf16(p0, p1);
      if (c * 16 + i == kPaceRelease - 1) release(pk[c][i]);
    }
  }
  float s0, s1, s2, s3;
  unpack2(sum_a, s0, s1);
  unpack2(sum_b, s2, s3);
  return (s0 + s1) + (s2 + s3);
}

// The K/V blocks of an item in the order they are loaded - the sorted union of the two query blocks' lists, each
// entry with two flags saying which tile uses it - for a role run by a single thread (producer, issuers).  The
// union is formed on the fly by a two-way merge of the lists; each list's next element is fetched one call early,
// so the global-load latency hides behind the current step.
template <bool kDense>
struct EntryStream {
  static constexpr int kEnd = 0x3fffffff;  // larger than any key block, below the flag bits
  const int32_t *l0, *l1;
  int n0, n1, i0, i1;
  int a, b, a_nx, b_nx;  // heads of the two lists and their successors (kEnd: exhausted)
  int e, m0, n_entries;  // dense
  bool tile1;
  __device__ __forceinline__ void init(const Item& it, const PrefillArgs& args) {
    m0 = it.m0;
    tile1 = it.tile1;
    n_entries = it.n_entries;
    e = 0;
    if (!kDense) {
      l0 = args.col_idx + it.base0;
      l1 = l0 + it.n0;
      n0 = it.n0;
      n1 = it.n1;
      i0 = i1 = 0;
      a = n0 > 0 ? __ldg(l0) : kEnd;
      a_nx = n0 > 1 ? __ldg(l0 + 1) : kEnd;
      b = n1 > 0 ? __ldg(l1) : kEnd;
      b_nx = n1 > 1 ? __ldg(l1 + 1) : kEnd;
    }
  }
  // the next entry of the stream; false when there is none
  __device__ __forceinline__ bool next(uint32_t* ent) {
    if (kDense) {
      if (e >= n_entries) return false;
      uint32_t x = static_cast<uint32_t>(e);
      if (e <= m0) x |= kFlag0;
      if (tile1) x |= kFlag1;
      ++e;
      *ent = x;
      return true;
    }
    const int J = min(a, b);
    if (J == kEnd) return false;
    uint32_t x = static_cast<uint32_t>(J);
    if (a == J) {
      x |= kFlag0;
      ++i0;
      a = a_nx;
      a_nx = i0 + 1 < n0 ? __ldg(l0 + i0 + 1) : kEnd;
    }
    if (b == J) {
      x |= kFlag1;
      ++i1;
      b = b_nx;
      b_nx = i1 + 1 < n1 ? __ldg(l1 + i1 + 1) : kEnd;
    }
    *ent = x;
    return true;
  }
};

// Items are taken in cost-sorted order by whichever CTA is free next (a device counter), so CTAs that run
// slower - the per-step time differs by a few per cent between SMs - simply take fewer of them.
template <bool kDense>
__global__ void __launch_bounds__(384, 1)
prefill_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
               const __grid_constant__ CUtensorMap tmap_v, const Dims d, const PrefillArgs a) {
  pdl_enter();
  extern __shared__ uint8_t smem_raw[];
  PrefillSmem& s = *reinterpret_cast<PrefillSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    s.abort_flag = 0;
    mbar_init(&s.q_full, 1);
    for (int i = 0; i < 4; ++i) mbar_init(&s.in_exp[i], 1);
    mbar_init(&s.q_free, 2);  // one arrival per issuer
    for (int i = 0; i < kStages; ++i) {
      mbar_init(&s.kv_full[i], 1);
      mbar_init(&s.kv_empty[i], 2);  // one arrival per issuer, whether or not its tile uses the block
    }
    for (int i = 0; i < 4; ++i) {
      mbar_init(&s.itm_full[i], 1);
      mbar_init(&s.itm_empty[i], 11);  // two issuers, eight softmax warps and the list prefetcher
    }
    for (int i = 0; i < 2; ++i)
      for (int h = 0; h < 2; ++h) {
        mbar_init(&s.s_full[i][h], 1);
        mbar_init(&s.p_ready[i][h], 128);
        mbar_init(&s.o_done[i][h], 1);
      }
    fence_mbar_init();
  }
  if (warp == 8) {
    tmem_alloc(&s.tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tm = s.tmem_base;
  volatile int* abort_flag = &s.abort_flag;
  // nothing is done when the selection stage reported an error (gate) or the lists failed validation (status)
  const int n_items = ((a.gate != nullptr && *a.gate != 0) || (!kDense && *a.status != 0)) ? 0 : a.n_items;

  // Register budget: the two softmax warpgroups hold a full 128-column row of S per thread; the third
  // warpgroup (producer, issuer, two idle warps) needs very few registers and gives the rest away.
  // (each role changes its own budget at the top of its branch)
  if (warp == 8) {
    // =============================================================== TMA producer
    reg_dealloc<kRegsOther>();
    if (lane == 0) {
      prefetch_tmap(&tmap_q);
      prefetch_tmap(&tmap_k);
      prefetch_tmap(&tmap_v);
    }
    if (lane == 0) {
      uint32_t ecount = 0;
      bool ok = true;
      for (int it_count = 0; ok; ++it_count) {
        const int qslot = it_count & 3;
        if (it_count >= 4) ok = mbar_wait(&s.itm_empty[qslot], ((it_count >> 2) - 1) & 1, abort_flag);
        if (!ok) break;
        int idx = n_items > 0 ? atomicAdd(a.next_item, 1) : -1;
        if (idx >= n_items) idx = -1;  // no more work: the others leave when they read this
        s.item_q[qslot] = idx;
        mbar_arrive(&s.itm_full[qslot]);
        if (idx < 0) break;
        const Item it = decode_item<kDense>(idx, d, a);
        EntryStream<kDense> rd;
        rd.init(it, a);
        if (it_count > 0) ok = mbar_wait(&s.q_free, (it_count - 1) & 1, abort_flag);
        if (!ok) break;
        mbar_arrive_expect_tx(&s.q_full, it.tile1 ? 65536u : 32768u);
        tma_load_3d(s.q[0][0], &tmap_q, &s.q_full, 0, it.h, it.m0 * kBlock);
        tma_load_3d(s.q[0][1], &tmap_q, &s.q_full, 64, it.h, it.m0 * kBlock);
        if (it.tile1) {
          tma_load_3d(s.q[1][0], &tmap_q, &s.q_full, 0, it.h, it.m1 * kBlock);
          tma_load_3d(s.q[1][1], &tmap_q, &s.q_full, 64, it.h, it.m1 * kBlock);
        }
        uint32_t ent;
        for (; ok && rd.next(&ent); ++ecount) {
          const int J = static_cast<int>(ent & kColMask);
          // loads 2*ecount (K) and 2*ecount + 1 (V) go to consecutive ring slots
#pragma unroll
          for (int which = 0; which < 2; ++which) {
            const uint32_t load = 2u * ecount + which;
            const int slot = load % kStages;
            const uint32_t use = load / kStages;
            if (use > 0) ok = mbar_wait(&s.kv_empty[slot], (use - 1) & 1, abort_flag);
            if (!ok) break;
            const CUtensorMap* tmap = which == 0 ? &tmap_k : &tmap_v;
            mbar_arrive_expect_tx(&s.kv_full[slot], 32768u);
            tma_load_3d(s.kv[slot][0], tmap, &s.kv_full[slot], 0, it.kvh, J * kBlock);
            tma_load_3d(s.kv[slot][1], tmap, &s.kv_full[slot], 64, it.kvh, J * kBlock);
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 9 || warp == 10) {
    // =============================================================== MMA issuers, one thread per tile
    reg_dealloc<kRegsOther>();
    constexpr uint32_t idesc_qk = umma_idesc_bf16(128, 64, false, false);   // S half: 128 x 64
    constexpr uint32_t idesc_pv = umma_idesc_bf16(128, 128, false, true);   // O: 128 x 128
    if (lane == 0) {
      const int t = warp - 9;
      const uint32_t flag_t = t == 0 ? kFlag0 : kFlag1;
      uint32_t ecount_base = 0;  // ring index of the item's first entry
      uint32_t p_count = 0;      // steps whose P has been consumed (phase of p_ready)
      bool ok = true;

      // Operand descriptors are built once; inside the loops only the 14-bit start-address field moves
      // (a compile-time offset per K step), so issuing an MMA costs two integer adds.
      // (an offset moves only the 14-bit start-address field in the descriptor's low word and cannot carry out
      // of it: a 32-bit add on the low word, not a 64-bit one - the issuing threads are on the critical path)
      auto desc_add = [](uint64_t desc, uint32_t off) {
        return (desc & 0xffffffff00000000ull) | static_cast<uint64_t>(static_cast<uint32_t>(desc) + off);
      };
      const uint64_t q_desc = umma_desc_sw128(smem_u32(s.q[t][0]), 0, 1024);
      // slot s of the ring starts 32 KB after slot s - 1: +2048 in the descriptor's address field
      const uint64_t k_desc0 = umma_desc_sw128(smem_u32(s.kv[0][0]), 0, 1024);      // K block: K-major B operand
      const uint64_t v_desc0 = umma_desc_sw128(smem_u32(s.kv[0][0]), 16384, 1024);  // V block: MN-major B operand
      const uint32_t s_tm = tm + t * 128, o_tm = tm + 256 + t * 128;

      // Every issuer observes every load of the ring in order and releases every slot once (a commit
      // behind the MMAs that read it, a plain arrival for a block only the other tile uses).  A slot is
      // therefore never refilled before both have seen it, so a phase parity can never be mistaken for
      // the one two refills earlier or later.
      uint32_t observed = 0;  // loads [0, observed) have been seen complete by this thread
      auto wait_next_load = [&]() {
        ok = ok && mbar_wait(&s.kv_full[observed % kStages], (observed / kStages) & 1, abort_flag);
        ++observed;
      };
      // observe and release the loads in [observed, load_end): blocks of the other tile
      auto skip_to = [&](uint32_t load_end) {
        while (observed < load_end && ok) {
          const int slot = observed % kStages;
          wait_next_load();
          if (ok) mbar_arrive(&s.kv_empty[slot]);
        }
      };
      // One step of this tile: ring index of its entry; whether it is the tile's last step (its diagonal).
      struct Step {
        uint32_t ec;
        bool last;
      };
      // S half h (keys 64 h .. 64 h + 63) = Q_t K_h^T: eight K steps of 16 dims, N = 64
      auto mma_qk_half = [&](const Step& st, int h) {
        const int slot = (2u * st.ec) % kStages;
        // key rows 64-127 of the block start 64 x 128 B further into each 64-dim half
        const uint64_t bd0 = desc_add(k_desc0, static_cast<uint32_t>(slot) * 2048u + static_cast<uint32_t>(h) * (8192u >> 4));
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          // K step kk: 64-column half kk / 4 (16 KB apart), 32 bytes per step inside the swizzle atom
          constexpr uint32_t kHalf = 16384 >> 4, kStep = 32 >> 4;
          const uint32_t off = (kk >> 2) * kHalf + (kk & 3) * kStep;
          umma_ss(s_tm + h * 64, desc_add(q_desc, off), desc_add(bd0, off), idesc_qk, kk > 0);
        }
        umma_commit(&s.s_full[t][h]);
        if (h == 1) {
          umma_commit(&s.kv_empty[slot]);
          if (st.last) umma_commit(&s.q_free);
        }
      };
      // O_t += P_h V_h: four steps of 16 keys; P_h (bf16) sits in columns 64 + 32 h .. of the tile's S region
      auto mma_pv_half = [&](const Step& st, int h, bool first) {
        const int slot = (2u * st.ec + 1u) % kStages;
        const uint64_t bd0 = desc_add(v_desc0, static_cast<uint32_t>(slot) * 2048u);
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) {
          const int kk = h * 4 + k4;
          // V block as the MN-major B operand: 16 keys per step = two groups of 8 key rows = 2048 B
          const uint32_t off = kk * (2048 >> 4);
          umma_ts(o_tm, s_tm + 64 + kk * 8, desc_add(bd0, off), idesc_pv, (kk > 0 || !first) ? 1u : 0u);
        }
        umma_commit(&s.o_done[t][h]);
        if (h == 1) umma_commit(&s.kv_empty[slot]);
      };

      for (int it_count = 0; ok; ++it_count) {
        const int qslot = it_count & 3;
        ok = mbar_wait(&s.itm_full[qslot], (it_count >> 2) & 1, abort_flag);
        if (!ok) break;
        const int idx = *reinterpret_cast<volatile int*>(&s.item_q[qslot]);
        mbar_arrive(&s.itm_empty[qslot]);
        if (idx < 0) break;
        const Item it = decode_item<kDense>(idx, d, a);
        ok = mbar_wait(&s.q_full, it_count & 1, abort_flag);
        if (!ok) break;
        if (t == 1 && !it.tile1) {
          // an item without a second tile: see its loads through (the K/V stream is block m0's list) and release Q
          const uint32_t n_stream = kDense ? it.n_entries : it.n0;
          skip_to(2u * (ecount_base + n_stream));
          if (ok) mbar_arrive(&s.q_free);
          ecount_base += n_stream;
          continue;
        }
        EntryStream<kDense> rd;
        rd.init(it, a);
        uint32_t e = 0;  // entries of the item's K/V stream walked so far
        // next step of this tile: walks the stream (flags only, never waits)
        auto find_next = [&](Step& st) {
          uint32_t ent;
          while (rd.next(&ent)) {
            ++e;
            if (ent & flag_t) {
              st.ec = ecount_base + e - 1;
              st.last = static_cast<int>(ent & kColMask) == (t == 0 ? it.m0 : it.m1);
              return true;
            }
          }
          return false;
        };

        Step cur, nx;
        bool have = find_next(cur);
        if (have) {
          skip_to(2u * cur.ec);
          wait_next_load();  // K of the first step
          if (!ok) break;
          tc_fence_after_sync();
          mma_qk_half(cur, 0);
          mma_qk_half(cur, 1);
        }
        // ---- steady state, two bursts per step.  The softmax hands P over in two halves; P lives in the
        // columns of S half B, so the columns of S half A are free as soon as P_A has been written (the
        // softmax has read both halves by then): the burst behind P_A is P_A V_A followed by the NEXT step's
        // Q K_A^T, the burst behind P_B is P_B V_B followed by the next Q K_B^T.  The softmax of the next step
        // therefore finds its first half waiting and its second half arrives while it works on the first:
        // neither the softmax nor the tensor pipe waits for a whole step of the other.
        bool first = true;
        while (have && ok) {
          const bool have_nx = find_next(nx);
          wait_next_load();  // V of this step (the load after its K)
          // The next K block may be waited for before this step's V is released only if it is at most two
          // entries ahead (a later one reuses the slot V sits in).
          const bool early = have_nx && nx.ec <= cur.ec + 2u;
          if (early) {
            skip_to(2u * nx.ec);
            wait_next_load();
          }
          ok = ok && mbar_wait(&s.p_ready[t][0], p_count & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          mma_pv_half(cur, 0, first);
          if (early) mma_qk_half(nx, 0);
          ok = mbar_wait(&s.p_ready[t][1], p_count & 1, abort_flag);
          if (!ok) break;
          ++p_count;
          tc_fence_after_sync();
          mma_pv_half(cur, 1, false);
          if (have_nx) {
            if (!early) {
              skip_to(2u * nx.ec);
              wait_next_load();
              if (!ok) break;
              tc_fence_after_sync();
              mma_qk_half(nx, 0);
            }
            mma_qk_half(nx, 1);
          }
          first = false;
          cur = nx;
          have = have_nx;
        }
        // blocks after this tile's diagonal belong to the other tile: walk the stream to its end and see them through
        {
          Step rest;
          while (find_next(rest)) {}
        }
        skip_to(2u * (ecount_base + e));
        ecount_base += e;
      }
    }
    __syncwarp();
  } else if (warp < 8) {
    // =============================================================== softmax / epilogue, one row per thread
    reg_alloc<kRegsSoftmax>();
    const int t = warp >> 2;                     // tile
    const int r = tid & 127;                     // row within the tile
    const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t s_addr = tm + lane_addr + t * 128;
    const uint32_t o_addr = tm + lane_addr + 256 + t * 128;
    uint32_t step_count = 0;  // steps of this tile so far (all items): phase of s_full / p_ready / o_done
    bool ok = true;
    // Pacing of the two tiles.  Warps w and w + 4 (the same rows of tile 0 and tile 1) sit on the same scheduler
    // and share its MUFU; left alone the tiles run in step, so both are in their exponentials at the same time
    // (the unit contended) and in their TMEM loads, maxima and stores at the same time (the unit idle).  Tile 1's
    // warp therefore flips a barrier of its scheduler when it enters a run of exponentials and again kPaceRelease
    // pairs into it, and tile 0's warp does not enter its own run while the barrier says "inside": tile 0 trails
    // tile 1 by a part of a run and each tile's exponentials overlap the other's loads and stores.  The wait is
    // a suspended try_wait that gives up after 2 us - it is a hint, never needed for progress, and nothing is
    // reported when it runs out (tile 1 may have no step at that time).
    uint64_t* in_exp = &s.in_exp[warp & 3];
    auto pace_enter = [&](float& pin) {
      if (t == 0) {
        // an odd phase is in progress <=> the wait for parity 1 has not completed
        if (!mbar_try_wait(in_exp, 1)) {
          const unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(in_exp, 1) && global_timer_ns() - t0 < 2000ull) {
          }
        }
        __syncwarp();
        asm volatile("" : "+f"(pin)::"memory");  // keeps the exponentials behind the wait
      }
      // (a separate test on purpose: written as the else of the branch above the same code measured 8 % slower)
      if (t == 1) {
        if (lane == 0) mbar_arrive(in_exp);
      }
    };
    auto pace_release = [&](uint32_t& pin) {
      if (t == 1) {
        asm volatile("" : "+r"(pin)::"memory");  // keeps the release where it stands among the exponentials
        __syncwarp();
        if (lane == 0) mbar_arrive(in_exp);
      }
    };
    // In-place rescale of the accumulator by 2^(m_used - m_new); every P*V issued so far must have completed.
    auto rescale_o = [&](float f) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t ov[32];
        tmem_ld_x32(o_addr + c * 32, ov);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * f);
        tmem_st_x32(o_addr + c * 32, ov);
      }
    };
    for (int it_count = 0; ok; ++it_count) {
      const int qslot = it_count & 3;
      ok = mbar_wait_warp(&s.itm_full[qslot], (it_count >> 2) & 1, abort_flag);
      if (!ok) break;
      const int idx = *reinterpret_cast<volatile int*>(&s.item_q[qslot]);
      __syncwarp();
      if (lane == 0) mbar_arrive(&s.itm_empty[qslot]);
      if (idx < 0) break;
      const Item it = decode_item<kDense>(idx, d, a);
      if (t == 1 && !it.tile1) continue;
      TileReader<kDense> rd;
      rd.init(it, a, t, lane);
      const int m_t = t == 0 ? it.m0 : it.m1;
      float m_used = 0.f, l_run = 0.f;
      bool first = true;
      // the key block of a step is looked up during the step before it (an item's first one here: the wait for its
      // first S covers the fetch), so the shuffle never sits between the arrival of S and the work on it
      int J_next = rd.get(0, lane);
      for (int i = 0; i < rd.n && ok; ++i) {
        const uint32_t ph = step_count & 1;
        const int J = J_next;
        const bool diag = (J == m_t);
        // Each 64-key half is one step of the online softmax.  The rescale decision is taken per warp
        // (the TMEM accesses are warp-collective): if any row of the warp outgrew its reference maximum by
        // more than the threshold, every row of the warp moves to its own current maximum.
        // ---------------- half A: keys 0-63
        ok = mbar_wait_warp(&s.s_full[t][0], ph, abort_flag);
        if (!ok) break;
        tc_fence_after_sync();
        uint32_t x[2][32];
        tmem_ld_x32(s_addr, x[0]);
        tmem_ld_x32(s_addr + 32, x[1]);
        if (i + 1 < rd.n) J_next = rd.get(i + 1, lane);  // under the TMEM loads
        tmem_ld_wait();
        float mx = (diag ? row_max<true>(x, r, 0) : row_max<false>(x, r, 0)) * d.scale_log2;
        if (first) {
          m_used = mx;  // key 0 is visible to every row, so this is finite
        } else if (__any_sync(0xffffffffu, mx > m_used + kRescaleThreshold)) {
          // the latest P*V issued is the second half of the previous step
          ok = mbar_wait_warp(&s.o_done[t][1], ph ^ 1u, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          const float m_new = fmaxf(m_used, mx);
          const float f = ex2(m_used - m_new);
          rescale_o(f);
          l_run *= f;
          m_used = m_new;
        }
        uint32_t pk[2][16];
        pace_enter(m_used);
        l_run += diag ? exp_pack<true>(x, r, 0, d.scale_log2, m_used, pk, pace_release)
                      : exp_pack<false>(x, r, 0, d.scale_log2, m_used, pk, pace_release);
        asm volatile("" : "+f"(l_run)::"memory");  // the run of exponentials ends here
        // ---------------- half B: keys 64-127.  Its logits leave TMEM before P_A goes into their columns.
        ok = mbar_wait_warp(&s.s_full[t][1], ph, abort_flag);
        if (!ok) break;
        tc_fence_after_sync();
        tmem_ld_x32(s_addr + 64, x[0]);
        tmem_ld_x32(s_addr + 96, x[1]);
        tmem_ld_wait();
        tmem_st_x16(s_addr + 64, pk[0]);
        tmem_st_x16(s_addr + 80, pk[1]);
        tmem_st_wait();
        tc_fence_before_sync();
        mbar_arrive(&s.p_ready[t][0]);
        mx = (diag ? row_max<true>(x, r, 64) : row_max<false>(x, r, 64)) * d.scale_log2;
        if (__any_sync(0xffffffffu, mx > m_used + kRescaleThreshold)) {
          // the latest P*V issued is the first half of this step
          ok = mbar_wait_warp(&s.o_done[t][0], ph, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          const float m_new = fmaxf(m_used, mx);
          const float f = ex2(m_used - m_new);
          rescale_o(f);
          l_run *= f;
          m_used = m_new;
        }
        pace_enter(m_used);
        l_run += diag ? exp_pack<true>(x, r, 64, d.scale_log2, m_used, pk, pace_release)
                      : exp_pack<false>(x, r, 64, d.scale_log2, m_used, pk, pace_release);
        asm volatile("" : "+f"(l_run)::"memory");  // the run of exponentials ends here
        tmem_st_x16(s_addr + 96, pk[0]);
        tmem_st_x16(s_addr + 112, pk[1]);
        tmem_st_wait();
        tc_fence_before_sync();
        mbar_arrive(&s.p_ready[t][1]);
        first = false;
        ++step_count;
      }
      if (!ok) break;
      // ---- epilogue: wait for the last P*V of this tile, normalise, store
      ok = mbar_wait_warp(&s.o_done[t][1], (step_count - 1) & 1, abort_flag);
      if (!ok) break;
      tc_fence_after_sync();
      const float inv = 1.0f / l_run;
      const size_t token = static_cast<size_t>(m_t) * kBlock + r;
      const bool in_range = token < static_cast<size_t>(d.n);  // the last block may be partial
      __nv_bfloat16* orow = a.o + (token * d.hq + it.h) * kHeadDim;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t ov[32];
        tmem_ld_x32(o_addr + c * 32, ov);
        tmem_ld_wait();
        uint4* dst = reinterpret_cast<uint4*>(orow + c * 32);
        if (in_range)
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          uint4 val;
          val.x = pack_bf16(__uint_as_float(ov[8 * g + 0]) * inv, __uint_as_float(ov[8 * g + 1]) * inv);
          val.y = pack_bf16(__uint_as_float(ov[8 * g + 2]) * inv, __uint_as_float(ov[8 * g + 3]) * inv);
          val.z = pack_bf16(__uint_as_float(ov[8 * g + 4]) * inv, __uint_as_float(ov[8 * g + 5]) * inv);
          val.w = pack_bf16(__uint_as_float(ov[8 * g + 6]) * inv, __uint_as_float(ov[8 * g + 7]) * inv);
          dst[g] = val;
        }
      }
      if (a.lse && in_range) a.lse[static_cast<size_t>(it.h) * d.n + token] = m_used * 0.6931471805599453f + logf(l_run);
      tc_fence_before_sync();
    }
  }
  else {
    // =============================================================== warp 11: pulls an item's lists into L2
    // The lists of a long prompt come from DRAM, and producer, issuers and softmax warps all walk them with
    // little look-ahead.  This warp touches every 128-byte line of an item's lists when the item starts (hints
    // only: nobody waits for them), so all but the first few entries are in L2 when they are asked for.
    reg_dealloc<kRegsOther>();
    bool ok = true;
    for (int it_count = 0; ok; ++it_count) {
      const int qslot = it_count & 3;
      ok = mbar_wait_warp(&s.itm_full[qslot], (it_count >> 2) & 1, abort_flag);
      if (!ok) break;
      const int idx = *reinterpret_cast<volatile int*>(&s.item_q[qslot]);
      __syncwarp();
      if (lane == 0) mbar_arrive(&s.itm_empty[qslot]);
      if (idx < 0) break;
      if (!kDense) {
        const Item it = decode_item<kDense>(idx, d, a);
        const char* lists = reinterpret_cast<const char*>(a.col_idx + it.base0);
        const long long bytes = static_cast<long long>(it.n0 + it.n1) * 4;
        for (long long off = static_cast<long long>(lane) * 128; off < bytes; off += 32 * 128)
          asm volatile("prefetch.global.L2 [%0];" ::"l"(lists + off));
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (tid == 0 && s.abort_flag) atomicExch(a.status, CRISP_ERR_DEVICE_TIMEOUT);
  if (warp == 8) tmem_dealloc(tm, 512);
}

// The lists of one item (query blocks m0 and, if the item is a pair, m0 + 1 of one head), checked before the
// attention kernel walks them.  The lists may come from the caller, so nothing about them is trusted: a row of
// query block m must hold between 1 and m + 1 entries inside the range `capacity` bounds, strictly ascending,
// none above m, the last one m itself (the diagonal block, which the attention kernel's Q hand-over relies on).
// Anything else marks the launch CRISP_ERR_BAD_LIST, and the attention kernel, which reads the status word,
// does no work at all.  One warp per item; it also enters the item into the histogram of the schedule's sort
// keys.
__global__ void __launch_bounds__(128)
check_lists_kernel(const Dims d, const int64_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
                   int* __restrict__ cost_hist, int n_pairs, int n_cost, int group_kv, const int* __restrict__ gate,
                   int* __restrict__ status, long long capacity, int rows_per_item, int* __restrict__ plain_order) {
  pdl_enter();
  if (gate != nullptr && *gate != 0) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // long lists first (the late query blocks), so that the launch ends on the short ones
  const int u = n_pairs - 1 - (blockIdx.x * 4 + warp), h = blockIdx.y;
  if (u < 0) return;
  const int m0 = rows_per_item * u, m1 = m0 + 1;
  const int64_t* rp = row_ptr + static_cast<size_t>(h) * (d.nb + 1);
  const int64_t s0 = rp[m0], e0 = rp[m0 + 1];
  const bool has1 = rows_per_item == 2 && m1 < d.nb;
  const int64_t e1 = has1 ? rp[m1 + 1] : e0;
  bool bad = s0 < 0 || e0 - s0 < 1 || e0 - s0 > m0 + 1 || e1 > capacity || (has1 && (e1 - e0 < 1 || e1 - e0 > m1 + 1));
  if (!bad) {
    // eight loads per lane in flight; an entry is compared with the one before it (the lane below, or the last
    // entry of the previous group of 32).  In range and strictly ascending; the last entry is the diagonal.
    constexpr int kInFlight = 8;
    auto check = [&](int64_t from, int64_t to, int m) {
      const int32_t* lst = col_idx + from;
      const int len = static_cast<int>(to - from);
      int prev_last = -1;
      for (int i0 = 0; i0 < len; i0 += 32 * kInFlight) {
        int c[kInFlight];
#pragma unroll
        for (int v = 0; v < kInFlight; ++v) {
          const int i = i0 + 32 * v + lane;
          c[v] = i < len ? __ldcs(lst + i) : 0x7fffffff;  // the padding passes the ascent test, not the range test
        }
#pragma unroll
        for (int v = 0; v < kInFlight; ++v) {
          const int i = i0 + 32 * v + lane;
          int before = __shfl_up_sync(0xffffffffu, c[v], 1);
          if (lane == 0) before = prev_last;
          bad = bad || (i < len && (static_cast<unsigned int>(c[v]) > static_cast<unsigned int>(m) || c[v] <= before));
          prev_last = __shfl_sync(0xffffffffu, c[v], 31);
        }
      }
      // (lists are not empty here: their lengths were checked above)
      if (lane == 0) bad = bad || __ldg(lst + len - 1) != m;
    };
    check(s0, e0, m0);
    if (has1) check(e0, e1, m1);
  }
  if (__any_sync(0xffffffffu, bad)) {
    if (lane == 0) atomicExch(status, CRISP_ERR_BAD_LIST);
    return;
  }
  if (plain_order != nullptr) {
    // every CTA of the attention kernel gets one item at most: any order will do, and no sort follows
    if (lane == 0) plain_order[h * n_pairs + u] = (n_pairs - 1 - u) * d.hq + h;
    return;
  }
  // sort key: KV head first, then decreasing cost (= tile steps = len(m0) + len(m1))
  if (lane == 0)
    atomicAdd(&cost_hist[(group_kv ? h / d.group : 0) * n_cost + (n_cost - 1 - static_cast<int>(e1 - s0))], 1);
}

// Counting sort of the items by (KV head, decreasing cost).  Grouping by KV head keeps the CTAs that
// run at the same time on the same K/V blocks (L2 reuse); sorting by cost inside a group lets the
// dynamic hand-out start the long lists (PE heads) before the short ones (VS heads).
// One thread per pair.  Every CTA first turns the histogram of its own segment (the keys of its KV head; all
// keys when the order is global) into first positions in shared memory - a segment holds a known number of
// items, so its base needs no other segment - and then places its items with one atomic each on a cursor array.
__global__ void __launch_bounds__(256)
sched_scatter_kernel(const Dims d, const int64_t* __restrict__ row_ptr, const int* __restrict__ cost_hist,
                     int* __restrict__ cursor, int* __restrict__ order, int n_pairs, int n_cost, int group_kv,
                     const int* __restrict__ gate, const int* __restrict__ status, int rows_per_item) {
  pdl_enter();
  extern __shared__ int first_pos[];  // [n_cost]
  __shared__ long long scratch[33];
  if (gate != nullptr && *gate != 0) return;
  if (*status != 0) return;  // a list failed validation: its row lengths cannot be trusted as histogram keys
  const int tid = threadIdx.x, h = blockIdx.y;
  const int seg = group_kv ? h / d.group : 0;
  const int* hist = cost_hist + static_cast<size_t>(seg) * n_cost;
  const int per = (n_cost + 255) / 256;
  const int b0 = min(tid * per, n_cost), b1 = min(b0 + per, n_cost);
  int local = 0;
  for (int i = b0; i < b1; ++i) local += hist[i];
  int run = static_cast<int>(block_exclusive_scan<256>(local, scratch, nullptr));
  for (int i = b0; i < b1; ++i) {
    first_pos[i] = run;
    run += hist[i];
  }
  __syncthreads();
  const int u = blockIdx.x * blockDim.x + tid;
  if (u >= n_pairs) return;
  const int64_t* rp = row_ptr + static_cast<size_t>(h) * (d.nb + 1);
  const int m0 = rows_per_item * u, mend = min(m0 + rows_per_item, d.nb);
  const int bin = n_cost - 1 - static_cast<int>(rp[mend] - rp[m0]);
  const int base = group_kv ? seg * n_pairs * d.group : 0;
  const int pos = base + first_pos[bin] + atomicAdd(&cursor[static_cast<size_t>(seg) * n_cost + bin], 1);
  order[pos] = (n_pairs - 1 - u) * d.hq + h;
}

struct PrefillWs {
  int* order;
  int* cost_hist;
  int* cursor;  // per sort key: items placed so far
  int n_cost;  // distinct cost values (0 .. 2 N_b + 1)
  int n_bins;  // n_cost per KV head
  size_t zero_bytes;  // header + histogram
};

PrefillWs carve(const Dims& d, void* ws, size_t* total) {
  PrefillWs w;
  uint8_t* base = static_cast<uint8_t*>(ws);
  size_t off = kWsHeader;
  const int n_pairs = d.nb;  // items per head at most (single-block items)
  // the histogram and the cursors sit directly behind the header: one memset clears all three
  w.n_cost = 2 * d.nb + 2;
  w.n_bins = w.n_cost * d.hkv;
  w.cost_hist = reinterpret_cast<int*>(base + off);
  off += align_up(sizeof(int) * static_cast<size_t>(w.n_bins), 256);
  w.cursor = reinterpret_cast<int*>(base + off);
  off += align_up(sizeof(int) * static_cast<size_t>(w.n_bins), 256);
  w.zero_bytes = off;
  w.order = reinterpret_cast<int*>(base + off);
  off += align_up(sizeof(int) * static_cast<size_t>(d.hq) * n_pairs, 256);
  *total = off;
  return w;
}

}  // namespace

size_t prefill_ws_bytes(const Dims& d) {
  size_t total;
  carve(d, nullptr, &total);
  return total;
}

int launch_prefill(const Dims& d, const void* q, const void* k, const void* v, const int64_t* row_ptr,
                   const int32_t* col_idx, void* ws, void* o, float* lse, cudaStream_t stream, const int* gate) {
  const bool dense = (row_ptr == nullptr);
  size_t total;
  PrefillWs w = carve(d, ws, &total);
  // status word, item counter and (sparse) the schedule histogram
  CRISP_CUDA_TRY(cudaMemsetAsync(ws, 0, dense ? kWsHeader : w.zero_bytes, stream), "prefill: clear status");
  CUtensorMap tq, tk, tv;
  int rc = make_tmap_bf16_nhd(&tq, q, d.n, d.hq);
  if (rc == CRISP_OK) rc = make_tmap_bf16_nhd(&tk, k, d.n, d.hkv);
  if (rc == CRISP_OK) rc = make_tmap_bf16_nhd(&tv, v, d.n, d.hkv);
  if (rc != CRISP_OK) return rc;

  PrefillArgs a;
  int dev = 0, n_sm = 0;
  CRISP_CUDA_TRY(cudaGetDevice(&dev), "prefill: device");
  CRISP_CUDA_TRY(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev), "prefill: SM count");
  // An item is a pair of adjacent query blocks, which share every K/V block in shared memory.  When the pairs do
  // not even fill the SMs, single blocks do better: twice the CTAs, and a block alone steps faster than a pair.
  a.rows_per_item = ((d.nb + 1) / 2) * d.hq < n_sm ? 1 : 2;
  a.n_pairs = (d.nb + a.rows_per_item - 1) / a.rows_per_item;
  a.n_items = a.n_pairs * d.hq;
  a.col_idx = col_idx;
  a.row_ptr = row_ptr;
  a.order = w.order;
  a.o = static_cast<__nv_bfloat16*>(o);
  a.lse = lse;
  a.status = static_cast<int*>(ws);
  a.gate = gate;
  a.next_item = static_cast<int*>(ws) + 16;  // inside the header that the memset above has just cleared
  // The schedule walks one KV head at a time, so the CTAs running at one moment stream the same K/V blocks.
  // Problems of only a few items per SM are ordered by cost alone instead: their K/V fit L2 anyway, and
  // the longest items of every head should start first.
  a.group_kv = 0;  // set below, once the SM count is known

  const int grid = a.n_items < n_sm ? a.n_items : n_sm;
  a.group_kv = a.n_items >= 16 * n_sm ? 1 : 0;
  const size_t smem = sizeof(PrefillSmem) + 1024;
  if (dense) {
    CRISP_CUDA_TRY(cudaFuncSetAttribute(prefill_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(smem)),
                   "prefill: smem attribute");
    CRISP_KERNEL("prefill_dense", stream, launch_pdl(prefill_kernel<true>, dim3(grid), dim3(384), smem, stream, tq, tk, tv, d, a));
  } else {
    // the lists are checked (and the items entered into the schedule's histogram) before anything walks them
    const long long capacity = static_cast<long long>(d.hq) * d.nb * (static_cast<long long>(d.nb) + 1) / 2;
    // with an SM for every item the schedule needs no sort: check_lists writes the order itself
    const bool one_item_per_cta = a.n_items <= n_sm;
    CRISP_KERNEL("check_lists", stream,
                 launch_pdl(check_lists_kernel, dim3((a.n_pairs + 3) / 4, d.hq), dim3(128), 0, stream, d, row_ptr, col_idx, w.cost_hist,
                            a.n_pairs, w.n_cost, a.group_kv, gate, a.status, capacity, a.rows_per_item,
                            one_item_per_cta ? w.order : nullptr));
    if (!one_item_per_cta) {
      const size_t scatter_smem = sizeof(int) * static_cast<size_t>(w.n_cost);
      if (scatter_smem > 48 * 1024)
        CRISP_CUDA_TRY(cudaFuncSetAttribute(sched_scatter_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            static_cast<int>(scatter_smem)),
                       "prefill: scatter smem attribute");
      CRISP_KERNEL("sched_scatter", stream,
                   launch_pdl(sched_scatter_kernel, dim3((a.n_pairs + 255) / 256, d.hq), dim3(256), scatter_smem, stream,
                       d, row_ptr, w.cost_hist, w.cursor, w.order, a.n_pairs, w.n_cost, a.group_kv, gate, a.status, a.rows_per_item));
    }
    CRISP_CUDA_TRY(cudaFuncSetAttribute(prefill_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(smem)),
                   "prefill: smem attribute");
    CRISP_KERNEL("prefill_sparse", stream, launch_pdl(prefill_kernel<false>, dim3(grid), dim3(384), smem, stream, tq, tk, tv, d, a));
  }
  CRISP_CUDA_TRY(cudaGetLastError(), "prefill: launch");
  return CRISP_OK;
}

}  // namespace crisp
