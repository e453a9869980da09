/*
 * curdkv.h -- C ABI of the B200 (sm_100a) implementation of CurDKV / AdaCurDKV
 * prefill-time KV-cache selection ("Value-Guided KV Compression for LLMs via
 * Approximated CUR Decomposition", Algorithm 1 and Sec. 3.2).
 *
 * For every (batch element, KV head) the library
 *   1. sketches the bf16 key and value matrices with a caller-supplied Gaussian
 *      matrix G and takes squared sketch-row norms (Alg. 1 (sketch and row norms)),
 *   2. multiplies key and value scores and normalises them per head (product and
 *      normalisation steps),
 *   3. keeps the sink and recent-window tokens and the top-scoring rest
 *      (sink, top-k and union steps), with a fixed budget per head or AdaCurDKV's layer-wide
 *      adaptive budgets (Sec. 3.2, "Adaptive budget allocation"),
 *   4. gathers the surviving rows into a compacted cache (gather step).
 *
 * General conventions
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer owned
 *     by the caller.  The library never allocates or frees device memory and
 *     never retains a pointer after a call returns.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     All work is enqueued on it; calls return without synchronising unless
 *     stated otherwise.  Such calls only launch kernels and memsets on the
 *     stream, so a sequence of them can be captured into a CUDA graph and
 *     replayed (curdkv_compress_host, which synchronises, cannot).
 *   - Return codes report errors the host can see (bad arguments, unsupported
 *     shapes, small workspace, launch failure).  Anomalies seen on the device
 *     (an out-of-range index, a bounded wait that ran out) are OR-ed into a
 *     status word at the start of the workspace; read it with
 *     curdkv_device_status().  No kernel traps or spins without limit.
 *   - Layers of a model may be folded into the batch axis: every batch element
 *     is an independent group of `kv_heads` problems.
 *   - Results are deterministic: identical inputs give bit-identical outputs.
 */
#ifndef CURDKV_H_
#define CURDKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum curdkv_status {
  CURDKV_OK = 0,
  CURDKV_ERR_INVALID_ARG = 1, /* NULL pointer, negative size, budget < 0, alpha outside [0,1] ... */
  CURDKV_ERR_UNSUPPORTED = 2, /* shape outside what the kernels handle (see curdkv_score)       */
  CURDKV_ERR_WORKSPACE = 3,   /* workspace smaller than curdkv_workspace_bytes()                 */
  CURDKV_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed                               */
  CURDKV_ERR_TIMEOUT = 5,     /* a bounded device-side wait ran out (from the status word)       */
  CURDKV_ERR_STATIC_LIMIT = 6 /* curdkv_score_static: shape needs more than its built-in scratch */
} curdkv_status;

/* Bits of the device status word (workspace[0], int32). */
#define CURDKV_DEV_TIMEOUT 0x1u   /* a pipeline wait gave up; results of that launch are invalid */
#define CURDKV_DEV_BAD_INDEX 0x2u /* an index outside [0, n) was skipped by the gather           */
#define CURDKV_DEV_CACHE_FULL 0x4u /* curdkv_cache_append dropped rows that exceeded the capacity */
#define CURDKV_DEV_NOT_SPD 0x8u   /* whiten = 1: a Gram matrix was not positive definite (raise ridge) */

/* Shape of one call: K and V are bf16 tensors addressed as
 *   K[b][h][j][c] = K_base[b*k_stride_b + h*k_stride_h + j*k_stride_n + c]
 * with strides in ELEMENTS, c contiguous; b < batch, h < kv_heads, j < n_max,
 * c < d.  Base addresses and all strides times 2 bytes must be multiples of 16.
 * (K in R^{g x n x d} of Alg. 1 with g = kv_heads, one such group per batch
 * element.) */
typedef struct curdkv_desc {
  int32_t batch;          /* independent (layer, sequence) groups                           */
  int32_t kv_heads;       /* g: KV groups per batch element                                 */
  int32_t q_heads;        /* query heads; a multiple of kv_heads (GQA), informational       */
  int32_t n_max;          /* rows allocated per (b, h)                                      */
  int32_t d;              /* head dimension                                                 */
  int32_t r;              /* sketch dimension (columns of G)                                */
  int64_t k_stride_b, k_stride_h, k_stride_n;
  int64_t v_stride_b, v_stride_h, v_stride_n;
  const int32_t* seqlens; /* device int32 [batch]: valid rows n_b (clamped to [0, n_max]),
                             or NULL when every sequence has n_max rows                     */
  int32_t score_mode;     /* 0: l = lK * lV (Alg. 1 (product step))  1: key only  2: value only
                             (ablation of App. C.3)                                         */
  int32_t use_projection; /* 1: sketch with G (Alg. 1 (sample G, project)); 0: raw squared row norms  */
  int32_t raw_scores;     /* 0: normalise per head (Alg. 1 (normalisation step)); 1: leave l^KV of the product step as
                             it is (head_sums is still written) -- what the generation-phase
                             cache stores, since a row's l^KV does not depend on other rows  */
  int32_t whiten;         /* 0: Alg. 1 as printed (||a_j G||^2 follows the row norms).
                             1: approximate the leverage scores ||U(j,:)||^2 of Eq. (row
                             leverage score): per (b, h) and tensor A in {K, V} over the valid
                             rows, M = A^T A + lambda I with lambda = ridge * trace(A^T A)/d,
                             M = L L^T (Cholesky), W = L^{-T} G, l_j = ||a_j W||^2; the rest of
                             Alg. 1 is unchanged.  Needs use_projection = 1, one shared G,
                             d = 128, r <= 64, n_max >= 128; reads K and V twice.          */
  double ridge;           /* whiten = 1 only: relative ridge >= 0 (1e-4 is a safe default;
                             0 needs n_b >= d and full column rank)                        */
} curdkv_desc;

/* Bytes of device workspace the calls below need for this shape (256-byte
 * aligned base required).  max_budget > 0 includes what curdkv_compress needs on
 * top of curdkv_score (three counters per head); max_budget = 0 sizes a workspace
 * for curdkv_score / curdkv_select / curdkv_compact alone.  `adaptive` is
 * reserved (it does not change the size today).  Returns 0 for an invalid
 * descriptor. */
size_t curdkv_workspace_bytes(const curdkv_desc* desc, int32_t max_budget, int32_t adaptive);

/* Alg. 1 (scoring steps): scores[b][h][j] = lK_j * lV_j / sum_j(lK_j * lV_j) with
 * lK_j = ||K[b][h][j] G||^2, lV_j = ||V[b][h][j] G||^2 (fp32 accumulation).
 *   G          fp32 [d][r] row-major shared by all heads (g_per_head = 0) or
 *              [kv_heads][d][r] (g_per_head = 1); the same G for K and V.
 *              Entries are expected ~N(0, 1/r) but any finite values work.
 *   scores     fp32 [batch][kv_heads][n_max]; entries j >= n_b are set to 0.
 *   head_sums  fp32 [batch][kv_heads]: the normaliser sum_j lK_j*lV_j.
 * Clears the device status word first.  Supported: d = 128, 1 <= r <= 64 with
 * projection; d % 8 == 0, d <= 1024 without.  Anything else returns
 * CURDKV_ERR_UNSUPPORTED and enqueues nothing. */
curdkv_status curdkv_score(const void* K, const void* V, const float* G, int32_t g_per_head,
                           const curdkv_desc* desc, float* scores, float* head_sums,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The paper has no counterpart of this call: it is curdkv_score for callers that
 * cannot give the library a workspace because they must not allocate device
 * memory -- code running where cudaMalloc is off limits (inside a host
 * framework that owns the whole memory pool, in a plugin that is handed only its
 * inputs and outputs, or late in a process that has already given all memory
 * away).  The scratch that curdkv_score takes from the caller (status words and
 * the per-tile partial sums of the head normaliser) lives here in an array built
 * into the library: 4 MiB + 256 bytes of device memory held by every GPU that
 * loads the library, until the process exits.
 *   - Same arguments and results (bit for bit) as curdkv_score, minus the
 *     workspace.
 *   - Limit: batch * kv_heads * ceil(n_max / 128) <= 262144 tiles (2^20 partial
 *     sums); larger shapes return CURDKV_ERR_STATIC_LIMIT and enqueue nothing.
 *   - desc->whiten = 1 is not available here (its Gram matrices and factors
 *     need 256 KiB and more of scratch per head): CURDKV_ERR_UNSUPPORTED.
 *   - status_flags: NULL, or a device uint32 that receives the device status
 *     word of this call (copied on the stream after the kernels).
 *   - The first call on each device looks up the array's device address (with
 *     that device current).  Make that first call outside any stream capture.
 *   - The call itself allocates and frees nothing, on the device or through any
 *     allocating library routine.
 *   - All calls on a device share the one array, and it keeps whatever the last
 *     call left in it; this call rewrites every word it later reads.  Two calls
 *     whose kernels overlap on the GPU (different streams, or different host
 *     threads without ordering) race on it: order them on one stream or with
 *     events. */
curdkv_status curdkv_score_static(const void* K, const void* V, const float* G, int32_t g_per_head,
                                  const curdkv_desc* desc, float* scores, float* head_sums,
                                  uint32_t* status_flags, void* cuda_stream);

/* Alg. 1 (sinks, top-k, union) (adaptive = 0) or AdaCurDKV (adaptive = 1).
 * Forced set of a sequence of n_b rows: the last `window` rows and the first
 * `num_sink` rows; if the budget cannot hold them all, the most recent window
 * rows come first, then sinks in index order.  Ties between equal scores go
 * to the lower token index (adaptive: lower head first, then lower index).
 * NaN or non-positive scores rank as 0.
 *   budget        k: rows kept per head, forced rows included; min(k, n_b) are kept
 *   head_budgets  adaptive = 0 only: NULL, or int32 [batch][kv_heads] per-head k
 *                 (each clamped to [0, budget])
 *   alpha         adaptive = 1 only: safeguard in [0,1]; every head keeps at least
 *                 min(max(floor(alpha*k), forced), min(k, n_b)) rows, the rest of the
 *                 layer total kv_heads*min(k, n_b) goes to the globally best rows
 *   workspace, workspace_bytes   reserved (not used today; NULL / 0 are accepted)
 *   idx           adaptive = 0: int32 [batch][kv_heads][budget], ascending token
 *                 index, unused tail = -1.  adaptive = 1: packed, head (b,h)
 *                 occupies idx[head_offsets[b*kv_heads+h] ...], ascending; capacity
 *                 batch*kv_heads*min(budget, n_max) entries.
 *   head_counts   int32 [batch][kv_heads]: rows kept per head
 *   head_offsets  int32 [batch*kv_heads + 1]: row of idx where each head starts.
 *                 adaptive = 1: exclusive prefix sums of head_counts (required);
 *                 adaptive = 0: p*budget, written only if not NULL
 * adaptive = 1 supports kv_heads <= 16. */
curdkv_status curdkv_select(const float* scores, const curdkv_desc* desc, int32_t budget,
                            const int32_t* head_budgets, int32_t num_sink, int32_t window,
                            int32_t adaptive, double alpha, int32_t* idx, int32_t* head_counts,
                            int32_t* head_offsets, void* workspace, size_t workspace_bytes,
                            void* cuda_stream);

/* Alg. 1 (gather step): K_out[row] = K[b][h][idx[...]], V_out likewise (byte copies).
 *   out_stride_h > 0  fixed layout: idx is [batch][kv_heads][idx_stride]; row t of
 *                     head (b,h) goes to output row (b*kv_heads+h)*out_stride_h + t
 *   out_stride_h = 0  packed layout: head (b,h) starts at row head_offsets[b*kv_heads+h]
 *                     of both idx and the outputs
 * Output rows are d contiguous bf16.  Rows beyond head_counts are left
 * untouched.  An index outside [0, n_b) is skipped and flagged in the status
 * word (workspace may be NULL: then it is only skipped). */
curdkv_status curdkv_compact(const void* K, const void* V, const curdkv_desc* desc,
                             const int32_t* idx, int64_t idx_stride, const int32_t* head_counts,
                             const int32_t* head_offsets, void* K_out, void* V_out,
                             int64_t out_stride_h, void* workspace, void* cuda_stream);

/* Alg. 1 (all steps) (or AdaCurDKV) in one call on device buffers: what curdkv_score,
 * curdkv_select and curdkv_compact do one after the other, with the same arguments,
 * the same outputs bit for bit (scores, head_sums, idx, head_counts, head_offsets,
 * gathered rows) and the default output layouts (adaptive = 0: idx
 * [batch][kv_heads][budget], K_out / V_out [batch][kv_heads][budget][d]; adaptive = 1:
 * packed).  With a fixed budget, one shared G, projection on, whiten off, d = 128,
 * r <= 32, n_max >= 128, no per-sequence lengths and at least one head per SM of the
 * device, the scoring kernel also normalises and selects: the heads whose last tile has been
 * written are handed, through one list served by all CTAs, to extra warps that run Alg. 1
 * normalisation and selection steps for them while the stream of K and V goes on, so the selection costs almost no
 * time of its own (a cooperative launch; it can still be captured into a CUDA graph), and the
 * gather is launched as that kernel's programmatic dependent: it copies the heads that are
 * already selected while the last heads, which finish streaming last, are being selected.  Other
 * shapes run the three steps in sequence, the selection kernel forming the head sums and
 * dividing on its first sweep instead of a separate normalisation pass.
 *   workspace   curdkv_workspace_bytes(desc, budget > 0 ? budget : 1, adaptive) bytes
 *   head_offsets  may be NULL when adaptive = 0
 * Enqueues kernels and memsets on the stream only. */
curdkv_status curdkv_compress(const void* K, const void* V, const float* G, int32_t g_per_head,
                              const curdkv_desc* desc, int32_t budget, const int32_t* head_budgets,
                              int32_t num_sink, int32_t window, int32_t adaptive, double alpha,
                              float* scores, float* head_sums, int32_t* idx, int32_t* head_counts,
                              int32_t* head_offsets, void* K_out, void* V_out, void* workspace,
                              size_t workspace_bytes, void* cuda_stream);

/* The whole path (Alg. 1 (all steps), or AdaCurDKV) for a cache that lives in HOST
 * memory: chunks of `chunk_batch` batch elements are copied to the device,
 * scored, selected and gathered, and the results copied back, double-buffered on
 * two internal streams so that copies overlap kernels.  Synchronous: returns when
 * every output is in host memory.  Pinned host buffers are needed for the overlap
 * (pageable ones work, serially).
 *   K_host, V_host   host bf16 [batch][kv_heads][n_max][d], dense (desc strides must say so)
 *   G_host           host fp32 [d][r] or [kv_heads][d][r]
 *   desc->seqlens    HOST int32 [batch] or NULL in this call
 *   K_out_host, V_out_host, idx_host, counts_host, offsets_host
 *                    host outputs with the layouts of curdkv_select / curdkv_compact
 *                    (offsets_host may be NULL when adaptive = 0)
 *   arena            device scratch of curdkv_host_arena_bytes() bytes, 256-byte aligned
 *   status_flags_host  NULL or host uint32: OR of the device status words of all chunks */
size_t curdkv_host_arena_bytes(const curdkv_desc* desc, int32_t budget, int32_t adaptive,
                               int32_t chunk_batch);
curdkv_status curdkv_compress_host(const void* K_host, const void* V_host, const float* G_host,
                                   int32_t g_per_head, const curdkv_desc* desc, int32_t budget,
                                   int32_t num_sink, int32_t window, int32_t adaptive, double alpha,
                                   void* K_out_host, void* V_out_host, int32_t* idx_host,
                                   int32_t* counts_host, int32_t* offsets_host, void* arena,
                                   size_t arena_bytes, int32_t chunk_batch, uint32_t* status_flags_host);

/* ---- Generation phase.  Sec. 3.2 notes that the method also applies while tokens are
 * generated, not only at prefill, and gives no procedure for it.  Reading used:
 * a cache holds, per (sequence, KV head), up to `capacity` rows of K and V with their
 * original token positions and their unnormalised scores l^KV (Alg. 1 (sketch, row norms, product)).
 * curdkv_cache_append scores newly generated rows and appends them;
 * curdkv_cache_compress applies Alg. 1 (normalisation, selection, gather) to the rows held at that moment
 * (sinks = positions < num_sink, window = the most recent `window` rows, the
 * best-scoring rest up to `budget`, ascending position order).  Incremental
 * compression keeps exactly the tokens a single application of Alg. 1 to the whole
 * history would keep.  All heads of a sequence hold the same number of rows.
 * Every pointer is a device pointer owned by the caller. */
typedef struct curdkv_cache {
  void* K;          /* bf16 [batch][kv_heads][capacity][d], dense                      */
  void* V;
  float* raw;       /* fp32 [batch][kv_heads][capacity]: l^KV of the held rows          */
  int32_t* pos;     /* int32 [batch][kv_heads][capacity]: token position of each row    */
  int32_t* count;   /* int32 [batch]: rows held per head; the caller zeroes it at start */
  int32_t* total;   /* int32 [batch]: tokens appended so far (= next position); idem    */
  int32_t capacity;
} curdkv_cache;

/* Workspace (256-byte aligned) for the two calls below: `t_max` = most rows appended
 * per head in one call, `budget` = largest budget compressed to.  0 = invalid. */
size_t curdkv_cache_workspace_bytes(int32_t batch, int32_t kv_heads, int32_t t_max,
                                    int32_t capacity, int32_t budget);

/* Appends K_new, V_new (bf16, described by desc_new exactly as in curdkv_score:
 * n_max = rows offered per head, seqlens = device int32 [batch] rows that are real,
 * or NULL) to the cache with their positions and l^KV under G.  Rows that would
 * exceed `capacity` are dropped and CURDKV_DEV_CACHE_FULL is set in the status word
 * (workspace[0]).  desc_new->raw_scores and ->score_mode are ignored (l^K * l^V). */
curdkv_status curdkv_cache_append(const curdkv_cache* cache, const void* K_new, const void* V_new,
                                  const float* G, int32_t g_per_head, const curdkv_desc* desc_new,
                                  void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Alg. 1 (normalisation, selection, gather) on the rows held in `in`; the kept rows, scores and positions go
 * to `out` (a different cache with capacity >= min(budget, in->capacity); the two
 * must not overlap), which also receives the counters.  Sequences holding at most
 * `budget` rows are copied unchanged.  desc supplies batch, kv_heads and d.
 * Forced rows are found by their POSITIONS (below num_sink; among the most recent
 * `window`), so the call also works on a cache that curdkv_cache_compress_inplace has
 * left unordered; the kept rows come out in the order of their slots in `in`, which is
 * ascending position order when `in` was ordered.  Requires num_sink + window <= budget. */
curdkv_status curdkv_cache_compress(const curdkv_cache* in, const curdkv_cache* out,
                                    const curdkv_desc* desc, int32_t budget, int32_t num_sink,
                                    int32_t window, void* workspace, size_t workspace_bytes,
                                    void* cuda_stream);

/* ---- Eviction loss (Lemma 1; the reconstruction-loss figure of the introduction):
 * how far the attention output moves when the cache is replaced by a selection,
 *   loss[b][h] = || softmax(scale Q K^T) V - softmax(scale Q K'^T) V' ||_F .
 * curdkv_attention_out computes O = softmax(scale * Q K^T) V for one cache (every
 * query row sees every valid key row: the question-after-context setting); call it
 * on the full cache and on the compacted one, then curdkv_eviction_loss.
 *   Q            bf16 [batch][kv_heads][q_rows][128] with element strides q_stride_*
 *                (the queries of a GQA group are stacked along q_rows)
 *   K, V, desc   the cache, as in curdkv_score (d = 128), unless head_offsets != NULL:
 *                then K and V are packed [packed_rows][128] arrays as curdkv_compact
 *                writes them for AdaCurDKV, head p starting at row head_offsets[p]
 *   head_rows    device int32 [batch*kv_heads] valid key rows per head, or NULL to use
 *                desc->seqlens / n_max (required with head_offsets)
 *   extra_zero_keys  NULL, or device int32 [batch*kv_heads]: that many further keys
 *                with logit 0 and value 0 take part in each softmax -- Lemma 1's K', V'
 *                keep the evicted rows as zero rows; NULL drops them, which is what a
 *                compressed cache computes
 *   scale        multiplies the logits (the paper writes softmax(QK^T): scale = 1)
 *   weight_split 1: the softmax weights enter the second product as bf16 pairs (hi + lo),
 *                so O agrees with an fp64 evaluation to about 1e-5 of its largest entry;
 *                0: as single bf16 values (a third fewer tensor-core products; O then
 *                agrees to about 2e-3 of its largest entry, each row of weights still
 *                sums to exactly the normaliser it is divided by)
 *   O            fp32 [batch][kv_heads][q_rows][128]; a head with no key rows gets 0
 * Online softmax in fp32 (exact up to rounding: no approximation of the maximum's
 * effect). */
size_t curdkv_attention_workspace_bytes(const curdkv_desc* desc);
curdkv_status curdkv_attention_out(const void* Q, int32_t q_rows, int64_t q_stride_b, int64_t q_stride_h,
                                   int64_t q_stride_n, const void* K, const void* V,
                                   const curdkv_desc* desc, const int32_t* head_rows,
                                   const int32_t* head_offsets, int64_t packed_rows,
                                   const int32_t* extra_zero_keys, float scale, int32_t weight_split,
                                   float* O, void* workspace, size_t workspace_bytes, void* cuda_stream);
/* loss[p] = ||O_full[p] - O_compressed[p]||_F and (if not NULL) ref_norm[p] = ||O_full[p]||_F
 * over elems_per_problem floats per problem; fixed summation order. */
curdkv_status curdkv_eviction_loss(const float* O_full, const float* O_compressed, int32_t problems,
                                   int64_t elems_per_problem, float* loss, float* ref_norm,
                                   void* cuda_stream);

/* The same compression inside one cache, for steady-state generation: the rows that are
 * kept stay where they are, and only survivors stored at or beyond slot min(budget, held)
 * move, into the slots the evicted rows leave below it (at most as many rows as were
 * evicted, instead of a copy of the whole cache).  Afterwards the cache holds its rows in no
 * particular order: `pos` tells which token each slot holds, and attention over the cache
 * does not depend on the order.  The kept SET is that of curdkv_cache_compress, except that
 * ties between equal scores go to the lower slot rather than the lower position.
 * Requires num_sink + window <= budget and capacity <= 204800. */
curdkv_status curdkv_cache_compress_inplace(const curdkv_cache* cache, const curdkv_desc* desc,
                                            int32_t budget, int32_t num_sink, int32_t window,
                                            void* workspace, size_t workspace_bytes, void* cuda_stream);

/* One generation step: what curdkv_cache_append followed by curdkv_cache_compress_inplace
 * does (same arguments, same resulting cache bit for bit, same status flags), in one kernel
 * after the scoring of the new rows.  The selection needs only scores and positions, so every
 * head first selects over its held rows' scores and the new rows' fresh ones; only then are
 * rows moved, each at most once: a surviving new row goes straight from K_new / V_new into its
 * final slot, a surviving held row beyond the new row count into a hole, and evicted new rows
 * are never copied.  Requires budget >= 1 and num_sink + window <= budget; capacities above
 * 36,864 rows run as the two calls. */
curdkv_status curdkv_cache_step(const curdkv_cache* cache, const void* K_new, const void* V_new,
                                const float* G, int32_t g_per_head, const curdkv_desc* desc_new,
                                int32_t budget, int32_t num_sink, int32_t window, void* workspace,
                                size_t workspace_bytes, void* cuda_stream);

/* GQA (Sec. 3.2): query head q uses KV head q / (q_heads / kv_heads).  Writes
 * kv_head_of_q int32 [q_heads] (device) so that attention consumers can index
 * the shared selection without replicating the compacted cache. */
curdkv_status curdkv_gqa_map(const curdkv_desc* desc, int32_t* kv_head_of_q, void* cuda_stream);

/* Optional expansion of a fixed-layout selection to the query heads (Sec. 3.2: the heads of a
 * GQA group share the keys and values of their group, hence its selection):
 *   idx_q[b][q][:] = idx[b][q / (q_heads / kv_heads)][:], counts_q[b][q] likewise.
 * idx int32 [batch][kv_heads][budget], idx_q int32 [batch][q_heads][budget],
 * counts_q int32 [batch][q_heads].  The compacted cache itself is never replicated. */
curdkv_status curdkv_gqa_expand(const curdkv_desc* desc, const int32_t* idx, const int32_t* head_counts,
                                int32_t budget, int32_t* idx_q, int32_t* counts_q, void* cuda_stream);

/* Copies the device status word to *host_flags (host pointer) after
 * synchronising the stream.  Returns CURDKV_ERR_TIMEOUT if the timeout bit is
 * set, CURDKV_OK otherwise (other bits are reported through *host_flags). */
curdkv_status curdkv_device_status(const void* workspace, uint32_t* host_flags, void* cuda_stream);

/* Self-test of the failure path (no counterpart in the paper).  Every wait inside the
 * pipelined kernels (TMA producer, MMA issuer, epilogue warps of the score, Gram and
 * attention kernels) is bounded: when its limit runs out the kernel sets
 * CURDKV_DEV_TIMEOUT, drains what it issued and returns.  This call runs that same
 * wait routine, with `limit_ns` (1 .. 10^9 nanoseconds) in place of the kernels'
 * 2 s, on a barrier that is never completed: one small kernel that comes back after
 * about limit_ns with CURDKV_DEV_TIMEOUT in the status word of `workspace` (at least
 * 256 bytes, 256-byte aligned; cleared first).  Nothing faults or traps, and the
 * stream stays usable: read the word with curdkv_device_status(). */
curdkv_status curdkv_selftest_bounded_wait(uint64_t limit_ns, void* workspace, void* cuda_stream);

/* The same for the one wait outside those kernels (no counterpart in the paper): inside
 * curdkv_compress the gather may start before the kernel that selects has ended, and each
 * of its CTAs then waits, bounded, for its head's ready flag.  This call launches that
 * gather for one head whose flag nothing ever sets, with `limit_ns` (1 .. 10^9) as the
 * limit: the kernel comes back after about limit_ns with CURDKV_DEV_TIMEOUT in the status
 * word of `workspace` (at least 512 bytes, 256-byte aligned; cleared first) and has read
 * and written nothing else. */
curdkv_status curdkv_selftest_gather_wait(uint64_t limit_ns, void* workspace, void* cuda_stream);

/* Profiling aid (no counterpart in the paper): asks the next curdkv_score or
 * curdkv_score_static call of THIS host thread to record the two cudaEvent_t
 * handles (passed as void*, either may be NULL) on its stream immediately
 * before and after its sketch kernel -- the kernel that streams K and V -- so
 * that a benchmark can time that kernel alone without a profiler.  The request
 * is cleared by that call.  With projection off or n_max < 128 the scores come
 * from a plain streaming kernel and nothing is recorded.  (Inside curdkv_compress
 * an event behind the kernel that scores and selects keeps the gather from
 * starting before that kernel has ended, which costs the call about 1 %.) */
curdkv_status curdkv_profile_next_score(void* start_event, void* stop_event);

/* Number of kernels this library has launched in this process so far. */
uint64_t curdkv_launch_count(void);

const char* curdkv_status_string(curdkv_status status);

#ifdef __cplusplus
}
#endif
#endif /* CURDKV_H_ */
