/*
 * crisp.h — C ABI of the B200 (sm_100a) implementation of CRISP's sparse-prefill attention path.
 *
 * One attention layer, all heads, one GPU.  The path is Algorithm 1 of the paper:
 *   crisp_route          proxy attention of the last query block + C_struct router + block scores
 *                        (Algorithm 2; Eq. 2; Algorithm 3 lines 3-5)
 *   crisp_select         sink-aware noise-floor selection (Algorithm 3 lines 6-12, Eq. 3-4), the
 *                        cumulative-gamma comparison rule (Algorithm 6), pooled estimation for PE heads
 *                        (Algorithm 4), and the expansion into per-query-block key-block lists
 *   crisp_sparse_prefill exact softmax attention over the listed blocks, causal (Eq. 1)
 *   crisp_dense_prefill  the same kernel over every causal block (the dense baseline)
 *
 * Conventions shared by every entry point
 *   - Tensors are contiguous, row major, bf16: Q and O are [seq_len, n_q_heads, 128]; K and V are
 *     [seq_len, n_kv_heads, 128].  Query head h reads KV head h / (n_q_heads / n_kv_heads).
 *   - All data pointers are DEVICE pointers owned by the caller.  The library never allocates or frees
 *     device memory; scratch memory is passed in as a workspace whose size crisp_workspace_bytes gives.
 *     Q, K, V, O and workspaces must be 16-byte aligned (256-byte recommended).
 *   - `cuda_stream` is a cudaStream_t (NULL = legacy default stream).  Calls only enqueue work on that
 *     stream and return; they never synchronise, except crisp_poll_device_status.
 *   - The return value is a crisp_status.  Host-side argument errors are reported immediately and
 *     nothing is launched.  Device-side conditions (capacity overflow, a bounded wait that gave up, index
 *     lists that break their rules) are recorded in the first word of the workspace and read back with
 *     crisp_poll_device_status.
 *   - Nothing throws, exits, traps or spins without a bound.
 *   - The library needs a CUDA device of compute capability 10.0; there is no CPU fallback.
 */
#ifndef CRISP_H_
#define CRISP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum crisp_status {
  CRISP_OK = 0,
  CRISP_ERR_INVALID_ARG = -1,    /* null pointer, non-positive size, inconsistent head counts, ...   */
  CRISP_ERR_UNSUPPORTED = -2,    /* head_dim != 128, block != 128, seq_len out of range, ...         */
  CRISP_ERR_WORKSPACE = -3,      /* workspace too small or misaligned                                */
  CRISP_ERR_CAPACITY = -4,       /* col_idx capacity too small for the selected blocks               */
  CRISP_ERR_CUDA = -5,           /* a CUDA runtime / driver call failed (see crisp_last_cuda_error)  */
  CRISP_ERR_DEVICE_TIMEOUT = -6, /* a bounded device-side wait gave up                               */
  CRISP_ERR_BAD_LIST = -7        /* row_ptr / col_idx given to crisp_sparse_prefill break the list rules */
} crisp_status;

/* Pattern labels written by crisp_route (Algorithm 2). */
#define CRISP_PATTERN_PE 0
#define CRISP_PATTERN_VS 1

/* Problem description: the inputs of Algorithm 1 plus the constants of Sections 3.2 and 4.3. */
typedef struct crisp_params {
  int32_t struct_size;   /* = sizeof(crisp_params); ABI guard                                        */
  int32_t seq_len;       /* n; 2 * block <= n <= 8192 * block (1,048,576); need not be a multiple of
                            `block`: N_b = ceil(n / block), the last block is partial (Section 4.3)  */
  int32_t n_q_heads;     /* H_q                                                                      */
  int32_t n_kv_heads;    /* H_kv; H_q % H_kv == 0 and H_q / H_kv <= 16                               */
  int32_t head_dim;      /* 128 only                                                                 */
  int32_t block;         /* B = 128 only (Section 4.3)                                               */
  int32_t sink_tokens;   /* w_sink: anchor keys j < w_sink (Eq. 2; paper value 128), 1..seq_len      */
  int32_t local_tokens;  /* w_local: anchor keys j >= n - w_local (Eq. 2; paper value 128)           */
  int32_t k_min_blocks;  /* minimum budget per direction in blocks (paper: 1024 tokens = 8), >= 0    */
  int32_t selector;      /* 0 = noise floor alpha (Algorithm 3); 1 = cumulative gamma (Algorithm 6);
                            2 = median noise floor (Appendix H: median instead of mean of the middle blocks) */
  int32_t force_pattern; /* 0 = route by C_struct; 1 = every head VS; 2 = every head PE              */
  float tau;             /* tau_proxy: VS iff C_struct >= tau (paper 0.2)                            */
  float alpha;           /* noise-floor multiplier (paper 1.0 / 1.25), >= 0                          */
  float gamma;           /* cumulative-mass target: PE heads always, VS heads when selector == 1     */
  float softmax_scale;   /* 0 => 1 / sqrt(head_dim)                                                  */
} crisp_params;

/* Library version: major * 10000 + minor * 100 + patch. */
int crisp_version(void);

/* Static string for a status code. */
const char* crisp_status_string(int status);

/* Text of the last CUDA error seen by this thread inside the library ("" if none). */
const char* crisp_last_cuda_error(void);

/*
 * Minimum workspace sizes in bytes for the three stages (any output pointer may be NULL).
 * The first 256 bytes of every workspace are a header whose first int32 is the device status word;
 * crisp_route / crisp_select / crisp_*_prefill clear it on entry (on the stream); before the first
 * such call on a workspace the word holds whatever the caller's allocation held.
 */
int crisp_workspace_bytes(const crisp_params* p, size_t* route_ws, size_t* select_ws, size_t* prefill_ws);

/*
 * Stage 1-3a (Algorithm 2; Algorithm 3 lines 3-5).  For every query head: the causal proxy attention
 * A_hat of the last `block` queries against all keys (never written to memory), then
 *   c_struct[h] = (1/block) sum_i sum_{j in anchors} A_hat[i, j]                              (Eq. 2)
 *   pattern[h]  = VS if c_struct[h] >= tau else PE (or the forced pattern)
 *   p_v[h, J]   = mass of key block J;  p_s[h, s] = mass of the diagonal band of block offset s,
 * both normalised to sum to 1.  Outputs: c_struct [H_q] f32, pattern [H_q] i32, p_v, p_s [H_q, N_b] f32.
 */
int crisp_route(const crisp_params* p, const void* q, const void* k, void* ws, size_t ws_bytes,
                float* c_struct, int32_t* pattern, float* p_v, float* p_s, void* cuda_stream);

/*
 * crisp_route for callers that are not able to obtain device memory at all.  (The paper has no
 * counterpart of this call; it exists for integration only and computes exactly what crisp_route does.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits or would fail, and that has no spare
 * buffer to lend as a workspace.  Typical cases are a plug-in invoked from inside a host application
 * that has already claimed the whole device for its own memory pool, and a latency-critical serving
 * loop whose rules forbid any call that may allocate or implicitly synchronise the device.
 *
 * How it works: the scratch that crisp_route takes as `ws` is replaced by one fixed array of
 * CRISP_ROUTE_STATIC_SCRATCH_BYTES bytes that is compiled into the library.  Every GPU that loads the
 * library carries this array from load time until the process exits, whether or not the call is used.
 * The caller passes the inputs and outputs only.  The call itself allocates nothing and frees nothing
 * (no cudaMalloc / cudaFree, no allocating library routine).
 *
 * Limits and rules
 *   - The problem must fit: crisp_workspace_bytes(p).route_ws <= CRISP_ROUTE_STATIC_SCRATCH_BYTES
 *     (4 MiB: for example 8192 tokens with 32 query heads, or 65536 tokens with 4, when seq_len is a
 *     multiple of `block`; other lengths need about 4/3 of that scratch, so 8191 tokens with 32 heads do not
 *     fit).  Anything larger is refused with CRISP_ERR_UNSUPPORTED before any work is enqueued, and
 *     crisp_last_cuda_error() says how many bytes would have been needed.
 *   - The first call on each device looks up the array's device address (with that device current) and
 *     remembers it for as long as the device's primary context lives (after cudaDeviceReset the remembered
 *     address is stale).  Make that first call during set-up, outside any stream capture.
 *   - All calls on one device share the one array.  Nothing of a previous call is ever read back (the
 *     status word is cleared, everything else is rewritten before use), but two calls that overlap in time
 *     on the same GPU - different streams, different threads - overwrite each other's scratch and give
 *     wrong results.  Serialise them (one stream, or an event between them).
 *   - device_status (optional, device pointer to one int32): receives the device status word of this
 *     call, CRISP_OK or CRISP_ERR_DEVICE_TIMEOUT, once the stream reaches that point.  There is no
 *     workspace pointer to hand to crisp_poll_device_status, so this is how the word is reported.
 * Outputs, layouts and all other conventions are those of crisp_route.
 */
#define CRISP_ROUTE_STATIC_SCRATCH_BYTES (4u << 20)
int crisp_route_static(const crisp_params* p, const void* q, const void* k, float* c_struct, int32_t* pattern,
                       float* p_v, float* p_s, int32_t* device_status, void* cuda_stream);

/*
 * Stage 3b-3c.  VS heads: per direction d in {v, s}, mu_d = (sum of the middle blocks of p_d)/(N_b - 2),
 * k_d = clip(#{p_d > alpha * mu_d}, k_min, N_b) (selector 0) or the smallest k whose top-k mass reaches
 * gamma (selector 1), S_d = top-k_d with ties to the lower index (Algorithm 3 / Algorithm 6).
 * PE heads: block means of Q and K, causal row softmax of their product, normalised by the total,
 * smallest prefix of the descending order whose mass reaches gamma (Algorithm 4).
 * Expansion: query block m of a VS head gets {0, m} u {J in S_v, J <= m} u {m-s, m-s-1 : s in S_s};
 * of a PE head {0, m} u {J : (m, J) selected}.
 *
 * Output is CSR over (head, query block): row_ptr [H_q, N_b + 1] int64 with global offsets into col_idx
 * (row_ptr[h][N_b] == row_ptr[h+1][0]); columns ascending, unique, all <= m, always containing 0 and m.
 * *nnz_needed (device int64) receives the total number of entries.  If it exceeds `capacity`, col_idx is
 * left untouched, the status word becomes CRISP_ERR_CAPACITY, and the lists must not be used.
 * q, k are read only for PE heads.
 */
int crisp_select(const crisp_params* p, const void* q, const void* k, const int32_t* pattern,
                 const float* p_v, const float* p_s, void* ws, size_t ws_bytes, int64_t* row_ptr,
                 int32_t* col_idx, int64_t capacity, int64_t* nnz_needed, void* cuda_stream);

/*
 * Stage 4 (Eq. 1).  O[t, h, :] = sum_j softmax_j(Q[t,h] . K[j,kv(h)] * scale) V[j,kv(h)] over the keys j <= t
 * of the key blocks listed for query block t / block.  Exact softmax over the kept keys; bf16 inputs,
 * fp32 accumulation, bf16 output.  lse (optional, [H_q, seq_len] f32) receives the natural-log
 * sum-exp of the kept scaled logits.  row_ptr / col_idx as produced by crisp_select, or built by the caller
 * to the same rules: row_ptr [H_q, N_b + 1] holds non-negative offsets into col_idx, at most
 * H_q N_b (N_b + 1) / 2, and col_idx holds at least row_ptr[H_q - 1][N_b] entries; the row of query block m
 * has between 1 and m + 1 entries, strictly ascending, all in [0, m], the last one m (the diagonal block).
 * The lists are checked on the device before they are used: if any row breaks a rule, nothing is computed,
 * O is left untouched and the status word of `ws` becomes CRISP_ERR_BAD_LIST.
 */
int crisp_sparse_prefill(const crisp_params* p, const void* q, const void* k, const void* v,
                         const int64_t* row_ptr, const int32_t* col_idx, void* ws, size_t ws_bytes, void* o,
                         float* lse, void* cuda_stream);

/*
 * Dense causal attention: crisp_sparse_prefill with every causal block listed (the baseline of Section 5).
 * Unlike the routed calls it accepts every seq_len from 1 to 8192 * block (sink_tokens and local_tokens are
 * not read); crisp_workspace_bytes reports route_ws = select_ws = 0 for seq_len < 2 * block.
 */
int crisp_dense_prefill(const crisp_params* p, const void* q, const void* k, const void* v, void* ws,
                        size_t ws_bytes, void* o, float* lse, void* cuda_stream);

/*
 * Comparison router (Algorithm 5, the FlexPrefill rule that C_struct replaces): the Jensen-Shannon distance
 *   jsd[h] = sqrt( 0.5 KL(a_hat || m) + 0.5 KL(a_bar || m) ),  m = (a_hat + a_bar) / 2,
 * between the per-query mean a_hat (= p_v of crisp_route, the block masses of the proxy map) and the pooled
 * estimate a_bar = Softmax(mean(Q_hat) . mean_block(K)^T * scale) over the N_b key blocks; natural logarithm,
 * terms of zero probability contribute 0.  pattern[h] = VS iff jsd[h] >= tau_jsd.  Not on the CRISP path: it
 * exists to measure how often the two routers agree.  Uses select_ws as scratch (block means of K), so it must
 * not overlap in time with crisp_select on the same workspace.  jsd [H_q] f32, pattern [H_q] i32.
 */
int crisp_route_jsd(const crisp_params* p, const void* q, const void* k, const float* p_v, void* select_ws,
                    size_t select_ws_bytes, float tau_jsd, float* jsd, int32_t* pattern, void* cuda_stream);

/*
 * Algorithm 1 in one call, with the context-length gate the paper recommends for deployments that serve
 * short prompts (Section 5.3, "Short contexts"): below dense_below_tokens the route and select launches take
 * longer than the skipped blocks would have.
 *   seq_len <  dense_below_tokens : crisp_dense_prefill only; the routing / selection outputs are not
 *                                   written and their pointers (and route_ws, select_ws) may be NULL.
 *   seq_len >= dense_below_tokens : crisp_route, crisp_select, crisp_sparse_prefill, enqueued back to back
 *                                   on the stream with no host synchronisation in between.
 * If the selected lists do not fit `capacity`, the attention kernels see the CRISP_ERR_CAPACITY word of
 * select_ws on the device and do nothing (O is left untouched); crisp_poll_device_status(select_ws)
 * reports it.  dense_below_tokens <= 0 disables the gate.  Arguments as in the staged calls.
 */
int crisp_forward(const crisp_params* p, const void* q, const void* k, const void* v, void* route_ws,
                  size_t route_ws_bytes, void* select_ws, size_t select_ws_bytes, void* prefill_ws,
                  size_t prefill_ws_bytes, float* c_struct, int32_t* pattern, float* p_v, float* p_s,
                  int64_t* row_ptr, int32_t* col_idx, int64_t capacity, int64_t* nnz_needed, void* o, float* lse,
                  int32_t dense_below_tokens, void* cuda_stream);

/*
 * A batch of independent sequences of different lengths, packed token-major (Algorithm 1 is defined per
 * sequence and per head; the paper's experiments use batch size 1, so the packing is this library's).
 * cu_seqlens is a HOST array of batch + 1 non-decreasing token offsets with cu_seqlens[0] = 0; sequence b holds
 * tokens cu_seqlens[b] .. cu_seqlens[b+1] - 1 of q, k, v, o; p->seq_len is ignored.  Every sequence is processed
 * exactly as crisp_forward would process it alone (same kernels, same results bit for bit), one after the other
 * on the stream; the three workspaces are reused and must be large enough for the longest sequence
 * (crisp_workspace_bytes with seq_len = that length).  A sequence shorter than max(dense_below_tokens, 2 * block)
 * gets dense attention (a sequence needs two blocks to be routed); an empty sequence is skipped.
 * With L_b the length of sequence b, N_b,b = ceil(L_b / block) and blk_off[b] = sum of N_b,b' over b' < b:
 *   c_struct, pattern  [batch][H_q]
 *   p_v, p_s           sequence b at element H_q * blk_off[b], laid out [H_q][N_b,b]
 *   row_ptr            sequence b at element H_q * (blk_off[b] + b), laid out [H_q][N_b,b + 1]; its values index
 *                      the sequence's own segment of col_idx
 *   col_idx            sequence b owns elements col_off[b] .. col_off[b+1] - 1, where
 *                      col_off[b] = floor(capacity * (causal blocks of the routed sequences before b) /
 *                      (causal blocks of all routed sequences)); capacity >= H_q * that total always suffices
 *   nnz_needed         [batch] (device), written for routed sequences only
 *   device_status      optional [batch][2] i32 (device): the status words of the selection stage
 *                      (CRISP_ERR_CAPACITY when the sequence's share of col_idx was too small; its rows of o are
 *                      then left untouched) and of the attention stage (CRISP_ERR_DEVICE_TIMEOUT), 0 when fine
 *   lse                optional; sequence b at element H_q * cu_seqlens[b], laid out [H_q][L_b]
 * crisp_varlen_layout returns blk_off and col_off (HOST arrays of batch + 1 int64) by the same rule, without
 * touching the GPU.  Entries of the outputs that belong to dense or empty sequences are not written.
 */
int crisp_varlen_layout(const crisp_params* p, const int64_t* cu_seqlens, int32_t batch, int64_t capacity,
                        int32_t dense_below_tokens, int64_t* blk_off, int64_t* col_off);
int crisp_forward_varlen(const crisp_params* p, const int64_t* cu_seqlens, int32_t batch, const void* q, const void* k,
                         const void* v, void* route_ws, size_t route_ws_bytes, void* select_ws, size_t select_ws_bytes,
                         void* prefill_ws, size_t prefill_ws_bytes, float* c_struct, int32_t* pattern, float* p_v,
                         float* p_s, int64_t* row_ptr, int32_t* col_idx, int64_t capacity, int64_t* nnz_needed,
                         int32_t* device_status, void* o, float* lse, int32_t dense_below_tokens, void* cuda_stream);

/*
 * Algorithm 1 for a layer whose Q, K, V and O live in HOST memory (the paper's Algorithm 1 is per head and has
 * no counterpart for the transfers: the chunking below is this library's).  The layer is cut into chunks of
 * kv_groups_per_chunk whole KV groups (a KV head with its H_q / H_kv query heads); chunk c is copied to the
 * device, run through crisp_route, crisp_select and crisp_sparse_prefill exactly as crisp_forward runs it, and
 * its output copied back, and the copies of one chunk overlap the kernels of another.  Every head's result is
 * bit for bit what crisp_forward gives for the whole layer.
 *   q_host, o_host [seq_len][H_q][128], k_host, v_host [seq_len][H_kv][128] bf16: HOST pointers.  Page-locked
 *     memory lets the copies overlap with the kernels; pageable memory works, but serialises them.
 *   kv_groups_per_chunk: 1 .. H_kv, a divisor of H_kv.
 *   stage: DEVICE buffer, 256-byte aligned, of at least crisp_forward_host_stage_bytes(p, kv_groups_per_chunk)
 *     bytes: two copies of a chunk's Q, K, V and O, the chunk's workspaces, routing outputs and lists (sized for
 *     all causal blocks, so the lists always fit).  Its contents after the call are unspecified.
 *   pattern_host (HOST, [H_q] i32) and nnz_host (HOST, one int64: blocks listed over all heads) are optional.
 * The kernels run on cuda_stream, the copies on two streams the library creates on first use (per device, kept
 * for the life of the process).  The call is synchronous: it returns when o_host is complete, with the first
 * error of any chunk (host-side, or a device status word: CRISP_ERR_DEVICE_TIMEOUT ...), else CRISP_OK.
 */
size_t crisp_forward_host_stage_bytes(const crisp_params* p, int32_t kv_groups_per_chunk);
int crisp_forward_host(const crisp_params* p, const void* q_host, const void* k_host, const void* v_host,
                       void* o_host, int32_t kv_groups_per_chunk, void* stage, size_t stage_bytes,
                       int32_t* pattern_host, int64_t* nnz_host, void* cuda_stream);

/*
 * Diagnostic (the paper has no counterpart): per-kernel device times of the stage calls, for benchmarks.
 * crisp_profile_enable(1) discards earlier records and switches recording on: from then on every kernel the
 * library launches is bracketed by two CUDA events on the caller's stream (the events are created on first use
 * and reused; this is host-side bookkeeping, but it is not meant for a production loop - it adds an event pair
 * per kernel and a process-wide lock).  crisp_profile_enable(0) switches it off and discards the records.
 * crisp_profile_read waits for the recorded kernels and returns, in launch order, up to max_records records:
 * names (HOST buffer of names_bytes bytes) receives the kernels' names separated by '\n', ms (HOST array of
 * max_records floats) their device times in milliseconds; *n_records = how many were returned.  Do not read
 * while a stream that holds recorded kernels is being captured.
 */
int crisp_profile_enable(int on);
int crisp_profile_read(char* names, size_t names_bytes, float* ms, int32_t max_records, int32_t* n_records);

/*
 * Diagnostic (the paper has no counterpart): exercises the library's failure-reporting path without any
 * failure.  Enqueues one tiny kernel that waits on a barrier nothing arrives at, with a wait limit of
 * `limit_ns` nanoseconds (1 .. 10,000,000); the wait runs out, a second role waiting with the normal limit is
 * released through the shared abort flag, the kernel records CRISP_ERR_DEVICE_TIMEOUT in the status word of
 * `ws` and returns by itself.  crisp_poll_device_status(ws) then reports that code, and the context stays
 * usable.  ws: device pointer, 16-byte aligned, at least 256 bytes; bytes 64..79 receive the two roles'
 * waiting times in nanoseconds (uint64 each).  limit_ns out of range: CRISP_ERR_INVALID_ARG, nothing launched.
 */
int crisp_selftest_bounded_wait(void* ws, size_t ws_bytes, int64_t limit_ns, void* cuda_stream);

/*
 * Synchronises `cuda_stream`, reads the status word at the start of `ws`, clears it and returns it
 * (CRISP_OK, CRISP_ERR_CAPACITY, CRISP_ERR_DEVICE_TIMEOUT or CRISP_ERR_BAD_LIST), or CRISP_ERR_CUDA if the
 * stream failed.
 */
int crisp_poll_device_status(void* ws, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* CRISP_H_ */
