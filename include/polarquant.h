/*
 * polarquant.h -- C ABI of the B200 (sm_100a) PolarQuant KV-cache library.
 *
 * The library implements the data-parallel hot path of PolarQuant ("Quantizing KV Caches
 * with Polar Transformation", arXiv 2502.02617): the KV-cache encoder of Algorithm 1
 * (random preconditioning, recursive polar transform, per-level angle codebooks, bit
 * packing) and decode attention over the packed cache (Eq. 3).
 *
 * General rules
 *   - Every function returns an int32 status: PQ_OK (0) or a negative PQ_ERR_* value.
 *     Nothing throws, aborts or traps.
 *   - "host" pointers are ordinary CPU memory, "dev" pointers are CUDA device memory of
 *     the current device.  The library allocates no device memory; every buffer belongs to
 *     the caller.  Device pointers must be 16-byte aligned.
 *   - State the library keeps, all of it per process: a call counter that tags the scratch of
 *     pq_decode_attention, a per-device note of which kernels have been configured (and, for
 *     pq_decode_attention_static, the device address of its built-in array, which every GPU
 *     that loads the library carries), the last CUDA error of each host thread, the analytic
 *     codebook pq_fit_codebooks_from_histograms starts from (computed at its first use), and the
 *     test hook of pq_debug_fail_next_wait.  All of it is updated atomically: host threads may call
 *     into the library concurrently as long as they do not share output buffers or scratch.
 *   - Device work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = the
 *     legacy default stream) and the call returns without synchronising.  The encode, append and
 *     decode-attention kernels are launched as programmatic dependents of whatever kernel precedes
 *     them in the stream: they may set up (barriers, tables from the caller's constant inputs) while
 *     that kernel finishes, and read K, V, q, the cache, the lengths and the workspace only after it
 *     has completed, so stream order holds for everything a caller can observe.  S_dev and
 *     tables_dev are the exception: they are read during that set-up, so they must not be written
 *     by the kernel that directly precedes the call in the stream (a copy, as in the binding, or any
 *     other operation in between is fine).
 *   - Problems that only the device can see (a sequence that would exceed `capacity`,
 *     an empty sequence in attention, non-finite inputs) are written to the caller's
 *     status words `status_dev` (int32[PQ_STATUS_WORDS], zero it before the first call):
 *       [0] first error code seen (0 = none)      [1] non-finite input elements seen
 *       [2] radii that saturated at the fp16 max  [3] 16-coordinate blocks that were
 *                                                     re-encoded by the float64 path
 *   - pq_make_rotation, pq_fit_codebooks, the encode / append calls and the attention calls open an NVTX
 *     range for the duration of the host call (a no-op unless a profiler is attached).
 *   - Row-vector convention of Algorithm 1: y = x . S, x_hat = y_hat . S^T; S is stored
 *     row-major [head_dim][head_dim] in float32.
 *   - Shapes: head_dim d in {16, 32, 64, 128}; L = 4 levels; bits (4,2,2,2) (Section 4.1);
 *     a block is 16 consecutive rotated coordinates and owns one fp16 radius.
 *   - Canonical code order of one vector (used by pq_unpack_codes): level-1 codes
 *     j = 0..d/2-1, then level 2 (d/4), level 3 (d/8), level 4 (d/16); angle j of level l
 *     is formed from entries 2j (cosine side) and 2j+1 (sine side) of level l-1.
 *   - GQA: query head h reads kv head h / (n_q_heads / n_kv_heads).
 */
#ifndef POLARQUANT_H_
#define POLARQUANT_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PQ_OK 0
#define PQ_ERR_INVALID_ARG (-1)  /* null pointer, non-positive size, bad head ratio */
#define PQ_ERR_UNSUPPORTED (-2)  /* head_dim / bits / dtype outside the supported set */
#define PQ_ERR_ALIGNMENT (-3)    /* a device pointer is not 16-byte aligned */
#define PQ_ERR_CAPACITY (-4)     /* a sequence would grow beyond `capacity` tokens */
#define PQ_ERR_CUDA (-5)         /* a CUDA runtime call failed (launch error) */
#define PQ_ERR_TIMEOUT (-6)      /* a bounded device-side wait gave up */
#define PQ_ERR_NONFINITE (-7)    /* inputs contained NaN or Inf */
#define PQ_ERR_EMPTY (-8)        /* attention over a sequence of length 0 */
#define PQ_ERR_SCRATCH (-9)      /* the problem needs more scratch than the built-in buffer holds */

#define PQ_DTYPE_F32 0
#define PQ_DTYPE_BF16 1

#define PQ_STATUS_WORDS 4
#define PQ_N_LEVELS 4
#define PQ_N_CENTROIDS 28  /* 16 + 4 + 4 + 4 */
#define PQ_N_BOUNDARIES 24 /* 15 + 3 + 3 + 3 */
#define PQ_HIST_MAX_BINS 1024 /* bins per level of pq_angle_histograms */
#define PQ_GENERAL_MAX_LEVELS 8 /* recursion depth of the pq_general_* entry points */

/* Human-readable name of a status code (static string, never NULL). */
const char* pq_status_string(int32_t status);

/* Text of the CUDA runtime error behind the calling thread's most recent PQ_ERR_CUDA ("" if none). */
const char* pq_last_cuda_error(void);

/* Tokens per cache token-block (a compile-time constant of the layout). */
int32_t pq_token_block(void);

/*
 * Random preconditioning matrix (Section 3.2 footnote; Section 4.1 "a random rotational
 * matrix"): a Haar-distributed orthogonal matrix obtained from the Householder QR of a
 * seeded Gaussian matrix with the signs of diag(R) folded into Q.  Computed in float64 on
 * the host, written as float32 to S_host[d*d] (row-major, y = x . S).  The same S is meant
 * to be shared by keys, values, all layers and all heads.
 */
int32_t pq_make_rotation(int32_t head_dim, uint64_t seed, float* S_host);

/*
 * Preconditioners without a dense random matrix (Section 3.2 asks only for an orthogonal S; its footnote
 * names fast transforms; Section 5's rows called "PolarQuant" without "-R" use none).  Written to
 * S_host[d*d] like pq_make_rotation; every entry point takes the result like any other S.
 *   kind = PQ_ROTATION_IDENTITY   S = I (signs_host is ignored and may be NULL)
 *   kind = PQ_ROTATION_HADAMARD   S = diag(signs) . H_d / sqrt(d), H_d the Sylvester Hadamard matrix
 *                                 (H_1 = [1], H_2n = [[H_n, H_n], [H_n, -H_n]]; head_dim a power of two);
 *                                 signs_host[d] holds +1 / -1 drawn by the caller
 * Returns PQ_ERR_INVALID_ARG for a NULL output, an unknown kind, a sign other than +1 / -1 or a missing sign
 * array, PQ_ERR_UNSUPPORTED for a head_dim that is not a power of two (Hadamard) or above 4096.
 */
#define PQ_ROTATION_IDENTITY 0
#define PQ_ROTATION_HADAMARD 1
int32_t pq_make_structured_rotation(int32_t head_dim, int32_t kind, const int8_t* signs_host, float* S_host);

/*
 * Angle codebooks (Algorithm 1 line 3, Eq. 4) for the analytic densities of Lemma 2:
 * level 1 uniform on [0, 2pi), level l >= 2 proportional to sin^(2^(l-1)-1)(2 psi) on
 * [0, pi/2].  Lloyd-Max iteration in float64 on the host.
 *   bits[4]            bits per level; only {4,2,2,2} is supported
 *   centroids_host     out, float64[PQ_N_CENTROIDS], ascending per level, levels concatenated
 *   boundaries_host    out, float64[PQ_N_BOUNDARIES], interior cell boundaries (midpoints)
 */
int32_t pq_fit_codebooks(const int32_t* bits, double* centroids_host, double* boundaries_host);

/*
 * Derived device tables (decision lines of the boundaries, cos/sin of the centroids in the
 * precisions the kernels use).  The codebook stays the paper's object; this is its compiled
 * form.  Any ascending centroids are accepted (e.g. a data-fitted codebook); boundaries are
 * the midpoints passed in.  tables_host must hold pq_tables_bytes() bytes; copy them to the
 * device unchanged and pass that pointer as `tables_dev`.
 */
int64_t pq_tables_bytes(void);
int32_t pq_build_tables(const double* centroids_host, const double* boundaries_host, void* tables_host);

/*
 * "Online" codebook (Section 4.1, Eq. 4 on the observed angles of one prompt and layer), in two steps.
 *
 * pq_angle_histograms: rotate the rows of K and V by S, take the angles of Algorithm 1's Polar and count them,
 * per level, in n_bins bins of equal width over the level's range ([0, 2 pi) at level 1, [0, pi/2] above).
 *   K_dev, V_dev       device, [total_tokens][n_kv_heads][head_dim] of `in_dtype`, strides in elements as for
 *                      pq_encode_kv (keys and values are counted together: one codebook serves both)
 *   n_bins             16 .. PQ_HIST_MAX_BINS
 *   hist_dev           device, uint64[PQ_N_LEVELS][n_bins], 8-byte aligned; counts are ADDED (zero it before the
 *                      first call; several calls accumulate, e.g. the chunks of one prompt)
 * Angles are formed in float32: an angle within about 1e-5 rad of a bin edge may be counted in the neighbouring
 * bin.  A 16-coordinate block with a non-finite rotated coordinate (any non-finite input of the row) is not
 * counted; the number of such blocks is added to status word 1 and PQ_ERR_NONFINITE is recorded.
 *
 * pq_fit_codebooks_from_histograms (host): per level, 1-D k-means (Lloyd's iteration) on the binned sample -- bin
 * centres weighted by their counts -- until no centroid moves: boundaries are the midpoints of adjacent centroids,
 * a bin belongs to the cell its centre lies in (a centre on a boundary: the lower cell), a centroid is the weighted
 * mean of its cell, and an empty cell keeps its centroid.  Distances are taken on the line, also at level 1.  The
 * paper seeds the clustering with k-means++; here it starts from init_centroids (NULL: the analytic codebook of
 * pq_fit_codebooks), so the result is a function of the histogram alone.
 *   hist_host          host, uint64[PQ_N_LEVELS][n_bins]
 *   init_centroids_host  host, float64[PQ_N_CENTROIDS] ascending per level, or NULL
 *   centroids_host, boundaries_host   out, as for pq_fit_codebooks; pass them to pq_build_tables
 * A level without any count keeps its initial centroids.
 */
int32_t pq_angle_histograms(int32_t head_dim, int32_t n_kv_heads, const float* S_dev, const void* K_dev,
                            const void* V_dev, int32_t in_dtype, int64_t token_stride, int64_t head_stride,
                            int32_t total_tokens, int32_t n_bins, uint64_t* hist_dev, int32_t* status_dev, void* stream);
int32_t pq_fit_codebooks_from_histograms(const uint64_t* hist_host, int32_t n_bins, const double* init_centroids_host,
                                         double* centroids_host, double* boundaries_host);

/* Size in bytes of the packed cache for `batch` sequences x n_kv_heads heads x (K and V),
 * each with room for `capacity` tokens (rounded up to whole token-blocks).  At d = 128 a
 * token costs exactly 62 bytes per head for K and 62 for V (Section 4.1: 3.875 bits per
 * coordinate); d < 64 pads the level-3/4 codes of a token to whole bytes.  Negative on
 * invalid arguments. */
int64_t pq_cache_bytes(int32_t head_dim, int32_t batch, int32_t n_kv_heads, int32_t capacity);

/* Scratch bytes pq_decode_attention needs (rotated queries, split partials, tickets). */
int64_t pq_workspace_bytes(int32_t head_dim, int32_t batch, int32_t n_q_heads, int32_t n_kv_heads,
                           int32_t max_len);

/*
 * Encode a prefill chunk of every sequence into the cache (Algorithm 1 lines 2 and 4, with
 * the codebooks fixed): rotate by S, L = 4 polar levels per 16-block, nearest centroid per
 * angle, fp16 block radii, bit packing.
 *   K_dev, V_dev       [total_tokens][n_kv_heads][head_dim] elements of `in_dtype`; element
 *                      (t, h, i) is at t*token_stride + h*head_stride + i (strides in elements)
 *   cu_seqlens_dev     int32[batch+1]: rows cu[b] .. cu[b+1]-1 belong to sequence b
 *                      (cu[0] = 0, cu[batch] = total_tokens)
 *   cache_lens_dev     int32[batch]: tokens already cached; the rows of sequence b are
 *                      written at positions lens[b] .. and lens[b] grows by its row count
 *   capacity           token capacity per sequence the cache was sized for; a sequence that
 *                      would exceed it is left untouched and PQ_ERR_CAPACITY is recorded
 * Angle decisions are taken in float32 with a certified margin; decisions inside the margin
 * are re-taken in float64, so codes match a float64 evaluation of Algorithm 1 unless the
 * angle lies within ~1e-13 rad of a boundary.
 */
int32_t pq_encode_kv(int32_t head_dim, int32_t n_kv_heads, const float* S_dev, const void* tables_dev,
                     const void* K_dev, const void* V_dev, int32_t in_dtype, int64_t token_stride,
                     int64_t head_stride, const int32_t* cu_seqlens_dev, int32_t batch,
                     int32_t total_tokens, void* cache_dev, int32_t* cache_lens_dev, int32_t capacity,
                     int32_t* status_dev, void* stream);

/*
 * Streaming generation step (Section 4: the stream (q_i, k_i, v_i)): encode one new token per
 * sequence at position lens[b] and increment lens[b].
 *   k_new_dev, v_new_dev   [batch][n_kv_heads][head_dim] contiguous, `in_dtype`
 */
int32_t pq_append_kv(int32_t head_dim, int32_t n_kv_heads, const float* S_dev, const void* tables_dev,
                     const void* k_new_dev, const void* v_new_dev, int32_t in_dtype, int32_t batch,
                     void* cache_dev, int32_t* cache_lens_dev, int32_t capacity, int32_t* status_dev,
                     void* stream);

/*
 * Decode attention over the packed cache (Eq. 3): for every sequence b and query head h,
 * softmax(K_hat q * scale)^T V_hat over the lens[b] cached tokens, K_hat / V_hat being
 * DeQuant (Algorithm 1) of the stored codes and radii.  The query is rotated once by S and
 * the result once by S^T; keys and values are decoded in the rotated basis only.
 *   q_dev          [batch][n_q_heads][head_dim] of `io_dtype` (PQ_DTYPE_BF16 or PQ_DTYPE_F32)
 *   out_dev        same shape and dtype; accumulation is float32
 *   max_len        host-side upper bound on lens[b] (used only to size the token splits)
 *   workspace_dev  pq_workspace_bytes(...) bytes of scratch; it need not be initialised (the split
 *                  counters inside are tagged with a per-call number) and need not be preserved;
 *                  two calls that overlap in time must not share it
 * A sequence with lens[b] = 0 yields zeros and records PQ_ERR_EMPTY.
 */
int32_t pq_decode_attention(int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads, const float* S_dev,
                            const void* tables_dev, const void* q_dev, int32_t io_dtype,
                            const void* cache_dev, const int32_t* cache_lens_dev, int32_t batch,
                            int32_t capacity, int32_t max_len, float scale, void* out_dev,
                            void* workspace_dev, int32_t* status_dev, void* stream);

/*
 * Attention of the last n_q positions of every sequence over the packed cache (Eq. 2 / Eq. 3 for a chunk of a
 * prefill or the drafted tokens of a speculative step).  The keys and values of those positions are already in
 * the cache (pq_encode_kv / pq_append_kv ran first); in the stream of Section 4 the i-th query attends to the
 * first i tokens, so query j (0-based) of a sequence sees the cached tokens t < lens[b] - (n_q - 1 - j), and
 * the last query sees all lens[b] of them.  n_q = 1 is pq_decode_attention.
 *   q_dev, out_dev   [batch][n_q][n_q_heads][head_dim] of `io_dtype`
 *   workspace_dev    pq_workspace_bytes(head_dim, batch * n_q, n_q_heads, n_kv_heads, max_len) bytes
 * A query that sees no token (lens[b] < n_q - j) yields zeros and records PQ_ERR_EMPTY.  At head_dim 128, chunks
 * of at least 128 rows (queries x query heads per kv head) run on a kernel that decodes every block of the cache
 * once for 128 -- two CTAs together: 256 -- rows and contracts on the tensor cores (no workspace is touched); so do
 * chunks of 32 to 127 rows when that is estimated to be faster (large batches, see pq_debug_fail_next_wait); shorter
 * chunks and other head_dims decode the cache once per query (the cost is n_q decode attentions).  batch * n_q
 * must not exceed 65535.
 */
int32_t pq_multi_query_attention(int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads, const float* S_dev,
                                 const void* tables_dev, const void* q_dev, int32_t io_dtype, const void* cache_dev,
                                 const int32_t* cache_lens_dev, int32_t batch, int32_t n_q, int32_t capacity,
                                 int32_t max_len, float scale, void* out_dev, void* workspace_dev, int32_t* status_dev,
                                 void* stream);

/*
 * pq_decode_attention for callers that cannot hand over scratch memory.  (The paper has no
 * counterpart; this is a packaging variant of the call above.)
 *
 * Some callers are not in a position to allocate device memory when they reach this call: code
 * running inside a region where the allocator must not be entered (a pre-sized serving loop with
 * a fixed memory plan, a plugin that is handed its tensors and nothing else, a caller replaying
 * a fixed sequence of launches).  For them the library carries its own scratch: a file-scope
 * device array of PQ_STATIC_SCRATCH_BYTES bytes that every GPU which loads the library keeps
 * until the process exits.  Arguments and results are those of pq_decode_attention without
 * `workspace_dev`.
 *   - Returns PQ_ERR_SCRATCH, and launches nothing, if pq_workspace_bytes(...) for these arguments
 *     exceeds PQ_STATIC_SCRATCH_BYTES (compare pq_static_scratch_bytes()).
 *   - The first call on each device looks up the device address of the array (a host-side query,
 *     no allocation); make that first call outside any stream capture.
 *   - Never calls cudaMalloc, cudaFree or any allocating routine.
 *   - All calls on a device share the one array.  It keeps the previous call's contents; nothing in
 *     it has to start at zero: the head_dim-128 kernel tags its split counters with the call's
 *     number and ignores counters of other calls, the other head_dims clear theirs in the call's
 *     first kernel.  Calls that may overlap on the GPU (different streams, no ordering) race on
 *     it: order them.
 */
#define PQ_STATIC_SCRATCH_BYTES (4 * 1024 * 1024)
int64_t pq_static_scratch_bytes(void);
int32_t pq_decode_attention_static(int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads, const float* S_dev,
                                   const void* tables_dev, const void* q_dev, int32_t io_dtype,
                                   const void* cache_dev, const int32_t* cache_lens_dev, int32_t batch,
                                   int32_t capacity, int32_t max_len, float scale, void* out_dev,
                                   int32_t* status_dev, void* stream);

/*
 * Test support: make the next launch of one kernel run its give-up path.  `which` = 1 arms the
 * tensor-core encoder behind pq_encode_kv (head_dim 128, bf16, >= 128 rows), 2 arms the head_dim-128
 * kernel behind pq_decode_attention, 4 the tcgen05 kernel behind pq_multi_query_attention (head_dim 128,
 * chunks that take that kernel, see below: its MMA-issuing thread gives up after two blocks, the other warps of
 * the CTA -- of the CTA pair -- follow, their rows are not written), 0 disarms.  In the armed launch the first bounded wait of one CTA
 * (the one that starts the first tile / the first non-empty sequence) is reported as failed although
 * what it waited for arrived: the CTA abandons its share of the work,
 * waits for its copies in flight, releases what it holds and records PQ_ERR_TIMEOUT in status word 0;
 * nothing on the device is left waiting and the next call runs normally.  (The paper has no
 * counterpart: it exercises the error handling of Section "General rules" without losing a copy.)
 * `which` = 3 is of another kind: the next pq_multi_query_attention call at head_dim 128 whose chunk has
 * 64 or more rows (queries x query heads per kv head) runs the register-fragment (mma.sync) kernel, which
 * no call reaches otherwise, so that it can be compared with the product path on the same inputs.  (The
 * tcgen05 kernel takes chunks of 128 rows and more, and chunks of 32 to 127 rows when its estimated time
 * -- kv heads x sequences CTA pairs walking max_len / 64 blocks -- is below that of one decode attention
 * per query; everything else runs the decode kernels with one (sequence, query) pair per unit.)
 */
int32_t pq_debug_fail_next_wait(int32_t which);

/*
 * Inspection (test support, not a hot path): unpack the first n_tokens positions of every
 * (sequence, kv head, K|V) into canonical order.
 *   codes_dev   uint8 [batch][n_kv_heads][2][n_tokens][15*d/16]   (index 2: 0 = K, 1 = V)
 *   radii_dev   fp16  [batch][n_kv_heads][2][n_tokens][d/16]
 */
int32_t pq_unpack_codes(int32_t head_dim, int32_t n_kv_heads, const void* cache_dev, int32_t batch,
                        int32_t capacity, int32_t n_tokens, uint8_t* codes_dev, void* radii_dev,
                        void* stream);

/* Inspection: DeQuant (Algorithm 1) of the first n_tokens positions, including the final
 * multiplication by S^T, with the decode arithmetic of the attention kernel.
 *   x_hat_dev   float32 [batch][n_kv_heads][2][n_tokens][d] */
int32_t pq_dequant_kv(int32_t head_dim, int32_t n_kv_heads, const float* S_dev, const void* tables_dev,
                      const void* cache_dev, int32_t batch, int32_t capacity, int32_t n_tokens,
                      float* x_hat_dev, void* stream);

/*
 * Paged cache (the packed layout of Section 4.1 behind a block table, as a serving engine keeps it): the cache is a
 * pool of n_pages pages; a page holds page_tokens tokens of every kv head -- [kv head][token-block of the page][K | V],
 * the layout of a contiguous cache of capacity page_tokens -- and sequence b's logical page p (positions
 * p * page_tokens ..) is physical page page_table[b * pages_per_seq + p].  A sequence may grow to
 * pages_per_seq * page_tokens tokens; only the table entries of pages it reaches are read.
 *   page_table_dev   device, int32[batch][pages_per_seq], 4-byte aligned; entries must name distinct pages for
 *                    distinct (sequence, logical page) -- the library cannot check that -- and lie in [0, n_pages):
 *                    a row whose page lies outside the pool is not written and its sequence does not grow (encode,
 *                    append), a reader reads page 0 instead; both record PQ_ERR_INVALID_ARG in the status words
 *   page_tokens      multiple of the token-block (pq_token_block()), of 128 at head_dim 128
 * The struct itself is read on the host during the call.  The *_paged entry points below are their contiguous
 * namesakes with `capacity` replaced by the paging; everything else (arguments, status words, tolerances) is the same,
 * and the codes, radii and attention outputs are those of a contiguous cache holding the same tokens.
 */
typedef struct pq_paging {
  const int32_t* page_table_dev;
  int32_t page_tokens;
  int32_t pages_per_seq;
  int32_t n_pages;
} pq_paging;

/* Bytes of a pool of n_pages pages. */
int64_t pq_paged_cache_bytes(int32_t head_dim, int32_t n_kv_heads, int32_t page_tokens, int32_t n_pages);
int32_t pq_encode_kv_paged(int32_t head_dim, int32_t n_kv_heads, const float* S_dev, const void* tables_dev,
                           const void* K_dev, const void* V_dev, int32_t in_dtype, int64_t token_stride,
                           int64_t head_stride, const int32_t* cu_seqlens_dev, int32_t batch, int32_t total_tokens,
                           void* cache_dev, int32_t* cache_lens_dev, const pq_paging* paging, int32_t* status_dev,
                           void* stream);
int32_t pq_append_kv_paged(int32_t head_dim, int32_t n_kv_heads, const float* S_dev, const void* tables_dev,
                           const void* k_new_dev, const void* v_new_dev, int32_t in_dtype, int32_t batch,
                           void* cache_dev, int32_t* cache_lens_dev, const pq_paging* paging, int32_t* status_dev,
                           void* stream);
int32_t pq_decode_attention_paged(int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads, const float* S_dev,
                                  const void* tables_dev, const void* q_dev, int32_t io_dtype, const void* cache_dev,
                                  const int32_t* cache_lens_dev, int32_t batch, const pq_paging* paging, int32_t max_len,
                                  float scale, void* out_dev, void* workspace_dev, int32_t* status_dev, void* stream);
int32_t pq_multi_query_attention_paged(int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads, const float* S_dev,
                                       const void* tables_dev, const void* q_dev, int32_t io_dtype, const void* cache_dev,
                                       const int32_t* cache_lens_dev, int32_t batch, int32_t n_q, const pq_paging* paging,
                                       int32_t max_len, float scale, void* out_dev, void* workspace_dev,
                                       int32_t* status_dev, void* stream);
int32_t pq_unpack_codes_paged(int32_t head_dim, int32_t n_kv_heads, const void* cache_dev, int32_t batch,
                              const pq_paging* paging, int32_t n_tokens, uint8_t* codes_dev, void* radii_dev, void* stream);
int32_t pq_dequant_kv_paged(int32_t head_dim, int32_t n_kv_heads, const float* S_dev, const void* tables_dev,
                            const void* cache_dev, int32_t batch, const pq_paging* paging, int32_t n_tokens,
                            float* x_hat_dev, void* stream);

/*
 * Partial attentions.  Softmax attention over a union of token sets is the weighted mean of the attentions over
 * the sets, with weights exp(lse_p - lse), lse_p = log sum_t exp(scale <q, k_t>) over set p (natural logarithm).
 * Two uses: the cached tokens of a sequence sharded over several GPUs (each GPU attends over its shard, the
 * (out, lse) pairs are gathered and merged on every GPU), and a cache whose most recent tokens are kept in 16 bits
 * (Section 5.3 keeps the generated tokens unquantised): compressed part and window are attended separately and merged.
 *
 * pq_decode_attention_lse: pq_decode_attention (paging == NULL: contiguous cache of `capacity` tokens; else the
 * paged cache and `capacity` is ignored) that also writes lse_dev, float32 [batch][n_q_heads].  A sequence of
 * length 0 yields zeros and lse = -inf and is NOT reported as PQ_ERR_EMPTY (an empty shard is legitimate).
 *
 * pq_merge_attention: parts_out_dev [n_parts][batch][n_q_heads][head_dim] of parts_dtype, parts_lse_dev float32
 * [n_parts][batch][n_q_heads] -> out_dev [batch][n_q_heads][head_dim] of out_dtype and, if not NULL, lse_out_dev.
 * Parts with lse = -inf are skipped; a row whose parts are all empty yields zeros, -inf and PQ_ERR_EMPTY.  Parts are
 * added in index order (bit-identical from run to run).  Use float32 parts: a part rounded to bf16 carries its
 * rounding into the merged output.
 *
 * pq_tail_attention: exact attention (Eq. 2) of one query per sequence over an uncompressed window,
 * k_tail_dev / v_tail_dev [batch][tail_capacity][n_kv_heads][head_dim] of kv_dtype, of which sequence b uses the
 * first tail_lens_dev[b] rows (16-byte aligned).  The window's tokens are cut into n_splits equal ranges, each
 * attended by its own thread blocks: out_dev holds n_splits parts, [n_splits][batch][n_q_heads][head_dim], and lse_dev
 * [n_splits][batch][n_q_heads], laid out as pq_merge_attention takes them (so the packed cache's part and the
 * window's parts can sit in one array and be merged by one call).  n_splits = 1 gives the attention over the whole
 * window; with lse_dev == NULL (n_splits = 1 only) an empty window records PQ_ERR_EMPTY.  Float32 arithmetic.
 */
int32_t pq_decode_attention_lse(int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads, const float* S_dev,
                                const void* tables_dev, const void* q_dev, int32_t io_dtype, const void* cache_dev,
                                const int32_t* cache_lens_dev, int32_t batch, int32_t capacity, const pq_paging* paging,
                                int32_t max_len, float scale, void* out_dev, float* lse_dev, void* workspace_dev,
                                int32_t* status_dev, void* stream);
int32_t pq_merge_attention(int32_t head_dim, int32_t n_q_heads, int32_t batch, int32_t n_parts, const void* parts_out_dev,
                           int32_t parts_dtype, const float* parts_lse_dev, void* out_dev, int32_t out_dtype,
                           float* lse_out_dev, int32_t* status_dev, void* stream);
int32_t pq_tail_attention(int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads, const void* q_dev, int32_t io_dtype,
                          const void* k_tail_dev, const void* v_tail_dev, int32_t kv_dtype, const int32_t* tail_lens_dev,
                          int32_t batch, int32_t tail_capacity, int32_t n_splits, float scale, void* out_dev,
                          float* lse_dev, int32_t* status_dev, void* stream);

/*
 * General recursion depth and bit tables.  Definition 1 recurses log2 d times and Section 4 counts
 * b_FPN + (d - 1) b bits per vector for b bits per angle; Section 4.1 stops at L = 4 with (4,2,2,2) bits, which the
 * entry points above implement at speed.  The pq_general_* entry points take any head_dim = 2^k <= 256, any
 * n_levels L with 2^L <= head_dim and any bits[l] in 1..6 for level l + 1 (a block is 2^L coordinates and owns one
 * fp16 radius), with plain kernels: the encoder works in float64 (codes are those of a float64 evaluation of
 * Algorithm 1: rotate, atan2, count the boundaries below the angle), attention in float32 with one thread block per
 * (sequence, kv head).  Reference speed, not the tuned path.
 *   codebooks      centroids float64[sum_l 2^bits[l]], boundaries float64[sum_l (2^bits[l] - 1)], levels concatenated,
 *                  ascending; pq_general_fit_codebooks gives the Lloyd-Max codebooks of the analytic densities
 *                  (Lemma 2); the device entry points take them as device arrays (8-byte aligned)
 *   cache          [batch][n_kv_heads][K | V][capacity][row_bytes]; a row holds, per level, the level's head_dim / 2^l
 *                  codes as one bit stream (least significant bit first, padded to a byte), padding to an even offset,
 *                  then the fp16 radii.  pq_general_sizes reports row_bytes and the counts.
 *   canonical code order (pq_general_unpack_codes): level 1 codes j = 0 .. d/2 - 1, then level 2, ...; angle j of
 *                  level l is formed from entries 2j (cosine side) and 2j + 1 of level l - 1
 * Status words, dtypes, strides, cu_seqlens and cache_lens behave as for pq_encode_kv / pq_decode_attention.
 */
typedef struct pq_general_config {
  int32_t head_dim;
  int32_t n_levels;
  int32_t bits[PQ_GENERAL_MAX_LEVELS];
} pq_general_config;

int32_t pq_general_sizes(const pq_general_config* cfg, int32_t* n_centroids, int32_t* n_boundaries, int32_t* n_codes,
                         int32_t* n_radii, int32_t* row_bytes);
int32_t pq_general_fit_codebooks(const pq_general_config* cfg, double* centroids_host, double* boundaries_host);
int64_t pq_general_cache_bytes(const pq_general_config* cfg, int32_t batch, int32_t n_kv_heads, int32_t capacity);
int32_t pq_general_encode_kv(const pq_general_config* cfg, int32_t n_kv_heads, const float* S_dev,
                             const double* boundaries_dev, const void* K_dev, const void* V_dev, int32_t in_dtype,
                             int64_t token_stride, int64_t head_stride, const int32_t* cu_seqlens_dev, int32_t batch,
                             int32_t total_tokens, void* cache_dev, int32_t* cache_lens_dev, int32_t capacity,
                             int32_t* status_dev, void* stream);
int32_t pq_general_decode_attention(const pq_general_config* cfg, int32_t n_q_heads, int32_t n_kv_heads, const float* S_dev,
                                    const double* centroids_dev, const void* q_dev, int32_t io_dtype, const void* cache_dev,
                                    const int32_t* cache_lens_dev, int32_t batch, int32_t capacity, float scale,
                                    void* out_dev, int32_t* status_dev, void* stream);
int32_t pq_general_unpack_codes(const pq_general_config* cfg, int32_t n_kv_heads, const void* cache_dev, int32_t batch,
                                int32_t capacity, int32_t n_tokens, uint8_t* codes_dev, void* radii_dev, void* stream);
int32_t pq_general_dequant_kv(const pq_general_config* cfg, int32_t n_kv_heads, const float* S_dev, const double* centroids_dev,
                              const void* cache_dev, int32_t batch, int32_t capacity, int32_t n_tokens, float* x_hat_dev,
                              void* stream);

#ifdef __cplusplus
}
#endif
#endif /* POLARQUANT_H_ */
