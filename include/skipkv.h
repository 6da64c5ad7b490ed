/*
 * skipkv.h -- C ABI of the B200 (sm_100a) hot path of SkipKV sentence-level KV eviction.
 *
 * Five operations, one per step of the path (paper: Section 4.1 "Skipping KV Storage with
 * Sentence-level Scoring", Section 4.2 "Skipping KV Generation with Adaptive Steering",
 * Algorithm 1 "Skipping KV Cache Storage"):
 *
 *   skipkv_score        sentence scores per (sequence, KV head)
 *   skipkv_select       which sentences survive under the KV budget
 *   skipkv_compact      in-place packing of the surviving K/V rows + range-table update
 *   skipkv_decode_attn  GQA decode attention over the ragged, compacted cache
 *   skipkv_steer        steering-vector add on the hidden state
 * and, beside them, the generation-space lookup table of the sentence penalty (skipkv_table_step)
 * with the score variant that reads it (skipkv_score_table), and the variants of select and compact that
 * retain exactly B tokens (skipkv_select_fill, skipkv_compact_fill), and the redundancy term over single
 * tokens (skipkv_token_redundancy) with the selection that uses it (skipkv_select_fill_red), the per-step append
 * (skipkv_append, skipkv_append_step) and its fusion with the attention (skipkv_decode_step), and the same steps
 * over a paged cache (skipkv_score_paged, skipkv_compact_paged, skipkv_decode_attn_paged,
 * skipkv_decode_step_paged).
 *
 * Conventions
 *   - Every pointer marked "device" is a CUDA device pointer; "host" is ordinary memory.
 *   - bf16 tensors are passed as void* (raw 16-bit patterns); head_dim must be 128.
 *   - Every call only enqueues work on `stream` (a cudaStream_t passed as void*; NULL is the
 *     default stream).  No call synchronises, allocates device memory or keeps state, except
 *     skipkv_status, which synchronises the stream to read one word back.
 *   - The caller owns every buffer.  Scratch memory comes from a caller-provided workspace of
 *     at least skipkv_workspace_bytes() bytes, 256-byte aligned, prepared once with
 *     skipkv_workspace_init().  One workspace serves one stream at a time.
 *   - Return value: 0 on success, a negative SKIPKV_ERR_* otherwise.  Nothing is enqueued
 *     when an argument check fails.  Device-side problems that cannot be seen at enqueue
 *     time (a bounded wait that ran out) are recorded in the workspace's status word.
 *   - No C++ exception crosses this boundary.
 *
 * Cache layout ("ragged slabs")
 *   One K and one V buffer per layer, bf16, rows of head_dim elements (256 bytes).  Sequence
 *   b owns rows [slab_off[b]*Hk, (slab_off[b]+cap[b])*Hk).  Inside that block KV head h owns
 *   cap[b] consecutive rows; the first kv_len[b][h] of them are live.  Row of (b, h, t):
 *   slab_off[b]*Hk + h*cap[b] + t.  There is no padding between sequences.
 *
 * Sentence tables (the cache-space range list M^(cs) of Algorithm 1), per (b, h):
 *   sent_off[b][h][0..max_sent]  token offsets, CSR: sentence i covers [sent_off[i], sent_off[i+1]);
 *                                sent_off[n_sent] == kv_len[b][h]
 *   sent_id [b][h][0..max_sent)  generation-space index of each sentence (the mapping Phi)
 *   n_sent  [b][h]
 */
#ifndef SKIPKV_H_
#define SKIPKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SKIPKV_OK               0
#define SKIPKV_ERR_INVALID_ARG (-1)  /* null pointer, negative size, inconsistent shape      */
#define SKIPKV_ERR_UNSUPPORTED (-2)  /* head_dim != 128, Hq % Hk != 0, group or window too big */
#define SKIPKV_ERR_WORKSPACE   (-3)  /* workspace null or misaligned                          */
#define SKIPKV_ERR_CUDA        (-4)  /* a CUDA runtime call failed; see skipkv_last_cuda_error */
#define SKIPKV_ERR_TIMEOUT     (-5)  /* reported by skipkv_status: a bounded device wait ran out */

/* Bits of the device status word (skipkv_status). */
#define SKIPKV_STATUS_COMPACT_TIMEOUT 0x1u  /* compaction hand-off wait ran out; rows of that slab are unspecified */
#define SKIPKV_STATUS_COPY_TIMEOUT    0x2u  /* a bulk copy did not complete within the wait limit */
#define SKIPKV_STATUS_BAD_TABLE       0x4u  /* a sentence table was inconsistent (offsets beyond cap, n_sent > max_sent) */

typedef struct {
    int32_t batch;        /* sequences                                                        */
    int32_t n_q_heads;    /* Hq                                                               */
    int32_t n_kv_heads;   /* Hk; Hq % Hk == 0, group n = Hq/Hk <= 8                           */
    int32_t head_dim;     /* must be 128                                                      */
    int32_t window;       /* observation window alpha (recent queries), n*alpha <= 512 and
                             alpha <= 4 * floor(128 / n) (at most four query blocks per group) */
    int32_t d_model;      /* hidden size of the steering add; multiple of 8                   */
    int32_t max_sent;     /* row stride of the sentence tables; every n_sent <= max_sent      */
    int32_t max_cap;      /* host-known upper bound of cap[b] (sizes grids and the workspace) */
    int64_t total_rows;   /* rows (of head_dim bf16) in each of the K and V buffers, host-known:
                             Hk * sum_b cap[b] for packed slabs; bounds the tiled copies         */
    const int64_t* slab_off; /* device [batch], in tokens                                     */
    const int32_t* cap;      /* device [batch], rows per (sequence, head)                     */
} skipkv_shape;

typedef struct {
    float   sigma;        /* importance/redundancy trade-off of the final score (paper: 0.1)  */
    float   tau;          /* similarity threshold of the redundant set (paper: 0.95..0.99)    */
    float   eps;          /* added to the norm of a pooled key                                */
    int32_t budget;       /* KV budget B in tokens per (sequence, head)                       */
    int32_t protect_tail; /* sentences touching the last protect_tail tokens are always kept  */
} skipkv_params;

/* Bytes of workspace needed for `shape` (host computation only). */
int skipkv_workspace_bytes(const skipkv_shape* shape, size_t* bytes);

/* Zero the workspace's counters and status word.  Once per workspace, and again after
 * skipkv_status reported an error.  ws: device. */
int skipkv_workspace_init(const skipkv_shape* shape, void* ws, void* stream);

/* Set how many times a bounded device wait polls before it gives up and records SKIPKV_STATUS_*_TIMEOUT in the
 * status word (every wait inside the kernels is bounded: a copy that never lands, or a hand-off another thread
 * block never makes, ends the wait instead of hanging the GPU).  polls = 0 restores the default (about four
 * million polls, seconds of waiting).  The value lives in the workspace, survives skipkv_workspace_init, and is
 * read by the kernels enqueued after this call on `stream`.  ws: device. */
int skipkv_set_wait_limit(void* ws, uint32_t polls, void* stream);

/* Self-check of the time-out path: enqueues one warp that waits, bounded by the workspace's wait limit, for an
 * event that never happens; when the wait runs out it records SKIPKV_STATUS_COPY_TIMEOUT like any kernel of this
 * library would, and returns.  Set a small limit first (with the default it spins for seconds).  ws: device. */
int skipkv_wait_probe(void* ws, void* stream);

/* Read and clear the device status word.  Synchronises `stream`.  *status_bits (host,
 * nullable) receives the SKIPKV_STATUS_* bits; returns SKIPKV_ERR_TIMEOUT if a wait ran out. */
int skipkv_status(void* ws, void* stream, uint32_t* status_bits);

/* Text of the last CUDA error seen by this library on the calling thread (host string). */
const char* skipkv_last_cuda_error(void);

/*
 * skipkv_score -- Section 4.1: token importance from the observation window (attention
 * equation, max over the heads of a group, mean over the window), sentence embeddings by mean
 * pooling, pairwise sentence similarity (Eq. "PSS"), the redundant set P, the redundancy term
 * (token-redundancy equation taken over sentences) and the final score (Eq. "I_final").
 * Per (b, h) slab with N = kv_len[b][h] live rows and S = n_sent[b][h] sentences:
 *   tok_imp[t]  = (1/alpha) sum_w max_{q in group h} softmax_t(q_win[b][q][w] . K[t] / sqrt(d))
 *   sent_imp[i] = mean of tok_imp over sentence i
 *   vbar_i      = mean of K rows of sentence i, divided by (its 2-norm + eps)
 *   G_ij        = vbar_i . vbar_j
 *   sent_red[i] = (1/S) sum_{j != i} exp(G_ji) / sum_{k != j} exp(G_jk)
 *   sent_lam[i] = max_{j > i} G_ij if that is > tau, else 0
 *   sent_score[i] = sigma*sent_imp[i] - (1-sigma)*sent_red[i] - sent_lam[i]
 * K: device bf16 (layout above, read only).  q_win: device bf16 [batch][Hq][window][128].
 * kv_len: device [batch][Hk].  sent_off / n_sent: device tables (read only).
 * tok_imp: device fp32, one value per cache row with the row indexing of K, nullable
 * (then it lives in the workspace).  sent_imp, sent_red, sent_lam, sent_score: device fp32
 * [batch][Hk][max_sent]; entries at i >= n_sent are not written.
 * shape->total_rows must be the exact number of rows of the K buffer (the tiled copies are bounded by
 * it).  The per-sentence sums are accumulated with floating-point atomics, so the last bits of the
 * scores may differ from run to run.  The kernels of one call, and the first kernel of a call after
 * the kernel before it on the stream, are launched as programmatic dependents: stream order holds.
 */
int skipkv_score(const skipkv_shape* shape, const skipkv_params* params, const void* K,
                 const void* q_win, const int32_t* kv_len, const int32_t* sent_off,
                 const int32_t* n_sent, float* tok_imp, float* sent_imp, float* sent_red,
                 float* sent_lam, float* sent_score, void* ws, void* stream);

/*
 * skipkv_select -- Section 4.1 (evict in increasing order of the final score until the cache
 * meets the budget B), at whole-sentence granularity.  Per slab: if kv_len <= budget keep
 * everything.  Otherwise rank sentences: those touching the last protect_tail tokens first (in
 * index order), then by (score descending, index ascending, exact fp32 comparison); walk the
 * ranking summing sentence lengths and keep the longest prefix whose total is <= budget (the
 * walk stops at the first sentence that does not fit).  Scores must not be NaN.
 * keep: device u8 [batch][Hk][max_sent] (1 = survives; entries >= n_sent set to 0).
 * kept_idx: device int32 [batch][Hk][max_sent], ascending sentence indices, nullable.
 * n_kept, new_len: device int32 [batch][Hk] (new_len = surviving tokens), nullable.
 */
int skipkv_select(const skipkv_shape* shape, const skipkv_params* params, const float* sent_score,
                  const int32_t* sent_off, const int32_t* n_sent, uint8_t* keep, int32_t* kept_idx,
                  int32_t* n_kept, int32_t* new_len, void* ws, void* stream);

/*
 * skipkv_compact -- Algorithm 1, eviction and post-eviction update (Eq. "after"): the rows of
 * the kept sentences move down, in their original order, to rows [0, new_len) of the same slab,
 * for K and for V, in place.  The range tables are rewritten: sent_off becomes the exclusive
 * prefix sum of the kept lengths (entries above the new n_sent are set to new_len), sent_id is
 * filtered (tail set to -1), n_sent and kv_len are updated; sentences with no surviving token
 * disappear.  index_map (device int32, one entry per cache row, row indexing of K, nullable):
 * index_map[row of (b,h,k)] = old token index of new token k, for k < new_len.
 * Rows at and beyond new_len are unspecified afterwards.  Moved rows are bit-identical copies.
 */
int skipkv_compact(const skipkv_shape* shape, void* K, void* V, const uint8_t* keep,
                   int32_t* sent_off, int32_t* sent_id, int32_t* n_sent, int32_t* kv_len,
                   int32_t* index_map, void* ws, void* stream);

/*
 * skipkv_decode_attn -- the attention equation of Section 4.1 with one query per head over the
 * live rows of each slab: out[b][q] = sum_t softmax_t(q[b][q] . K[t] / sqrt(d)) V[t] for
 * t < kv_len[b][q / n]; fp32 accumulation, bf16 result; kv_len == 0 gives zeros.
 * q, out: device bf16 [batch][Hq][128].  If hidden is non-null the steering add of
 * skipkv_steer is performed on it by the same launch (arguments as below).
 */
int skipkv_decode_attn(const skipkv_shape* shape, const void* q, const void* K, const void* V,
                       const int32_t* kv_len, void* out, void* hidden, const void* steer_vec,
                       const float* alpha, const uint8_t* flag, void* ws, void* stream);

/*
 * skipkv_steer -- Section 4.2: H <- H + alpha_t * v for the sequences whose current token is a
 * delimiter.  hidden: device bf16 [batch][d_model], in place.  steer_vec: device bf16
 * [d_model].  alpha: device fp32 [batch] (alpha_0 + gamma*N_o, computed by the caller).
 * flag: device u8 [batch], rows with 0 are untouched.  One fp32 fused multiply-add per
 * element, rounded to nearest even bf16.
 */
int skipkv_steer(int32_t batch, int32_t d_model, void* hidden, const void* steer_vec,
                 const float* alpha, const uint8_t* flag, void* stream);

/*
 * skipkv_append -- pre-eviction bookkeeping of Algorithm 1 for one decode step: writes the new
 * K/V row of every (b, h) at position kv_len[b][h] and increments kv_len.  k_new, v_new:
 * device bf16 [batch][Hk][128].  A slab that is already full (kv_len == cap) is left
 * unchanged and SKIPKV_STATUS_BAD_TABLE is raised in the status word of ws.
 */
int skipkv_append(const skipkv_shape* shape, void* K, void* V, const void* k_new, const void* v_new,
                  int32_t* kv_len, void* ws, void* stream);

/*
 * skipkv_table_step -- Section 4.1 "Sentence Similarity Score" and the lookup table T of Eq.
 * "sentence-score-input", maintained one decode step at a time.  A sentence embedding is the mean of
 * the LAST-LAYER hidden-state rows of the sentence's tokens (delimiter included), divided by
 * (its 2-norm + eps); the similarity of two sentences is the dot product of their embeddings (Eq. "PSS");
 * T[i] = max over later sentences j of that similarity when it exceeds tau, else 0 (the earlier sentence
 * of a redundant pair is flagged, the later one kept).  Per sequence b this call
 *   - adds hidden_last[b] to the running sum of the open sentence (acc, acc_count);
 *   - if flag[b] != 0 (the token is a delimiter) closes the sentence: stores its embedding at
 *     emb[b][n_gen_sent[b]], sets T[b][that index] = 0, increments n_gen_sent[b], clears the running sum,
 *     writes the index to closed[b], and raises T[b][i] to the similarity with every earlier sentence i
 *     whose similarity exceeds tau and the current entry;
 *   - otherwise writes closed[b] = -1.
 * After any number of steps T equals the one-shot definition over the closed sentences.
 * hidden_last: device bf16 [batch][d_model] (read only).  flag: device u8 [batch].
 * State, caller-owned, zero before the first step: acc device fp32 [batch][d_model], acc_count device int32
 * [batch], n_gen_sent device int32 [batch].  emb: device fp32 [batch][max_gen_sent][d_model].
 * lam_table: device fp32 [batch][max_gen_sent] (entries at and beyond n_gen_sent are not meaningful).
 * closed: device int32 [batch] (output).  status: device uint32, nullable: SKIPKV_STATUS_BAD_TABLE is OR-ed
 * in when a sentence closes with n_gen_sent == max_gen_sent (that sentence is dropped).
 * d_model: multiple of 8, at most 16384; hidden_last, acc and emb 16-byte aligned.
 */
int skipkv_table_step(int32_t batch, int32_t d_model, int32_t max_gen_sent, const void* hidden_last,
                      const uint8_t* flag, float* acc, int32_t* acc_count, float* emb, int32_t* n_gen_sent,
                      int32_t* closed, float* lam_table, float tau, float eps, uint32_t* status, void* stream);

/*
 * skipkv_score_table -- skipkv_score with the sentence penalty taken from the lookup table through the
 * mapping Phi of Eq. "sentence-score-cache" instead of the pooled keys:
 *   sent_lam[i] = lam_table[b][sent_id[b][h][i]] if 0 <= sent_id[b][h][i] < table_len, else 0.
 * Importance, redundancy and the final score are those of skipkv_score.  sent_id: device table (read
 * only).  lam_table: device fp32 [batch][table_len] (row stride table_len), e.g. the table kept by
 * skipkv_table_step with table_len = max_gen_sent.  Other arguments, limits and launch behaviour as
 * skipkv_score.
 */
int skipkv_score_table(const skipkv_shape* shape, const skipkv_params* params, const void* K,
                       const void* q_win, const int32_t* kv_len, const int32_t* sent_off,
                       const int32_t* sent_id, const int32_t* n_sent, const float* lam_table,
                       int32_t table_len, float* tok_imp, float* sent_imp, float* sent_red, float* sent_lam,
                       float* sent_score, void* ws, void* stream);

/*
 * skipkv_select_fill, skipkv_compact_fill -- Section 4.1 taken to exactly B survivors (tokens leave in
 * increasing order of the final score until the cache meets the budget).  skipkv_select_fill keeps whole
 * sentences as skipkv_select does; the first sentence of the ranking that does not fit (the cut sentence)
 * then keeps its slack = B - kept tokens of largest tok_imp -- redundancy and penalty are constant inside a
 * sentence, so there the final-score order is the importance order; equal values: the earlier token.  That
 * sentence gets keep = 2 and its tokens are flagged in tok_keep (device u8, one byte per cache row with the
 * row indexing of K; only the bytes of a cut sentence are written or meaningful).  new_len is B for every
 * slab that was over the budget (when slack is 0 nothing is cut and the result is that of skipkv_select).
 * tok_imp: device fp32 per cache row as written by skipkv_score, or NULL to use the copy that the last
 * skipkv_score call left in this workspace.  Other arguments as skipkv_select.
 *
 * skipkv_compact_fill is skipkv_compact for such a selection: a sentence with keep = 2 survives with its
 * flagged tokens only, in order; ranges follow Eq. "after" (b <- min{k : p_k >= b}, e <- max{k : p_k <= e}
 * over the survivor list p), so the cut sentence stays in the tables with its shortened length, and
 * index_map names each survivor's old token index.  At most 4 sentences with keep = 2 per slab (more:
 * SKIPKV_STATUS_BAD_TABLE and that slab is left unmoved).  tok_keep is read only.
 */
int skipkv_select_fill(const skipkv_shape* shape, const skipkv_params* params, const float* sent_score,
                       const float* tok_imp, const int32_t* sent_off, const int32_t* n_sent, uint8_t* keep,
                       uint8_t* tok_keep, int32_t* kept_idx, int32_t* n_kept, int32_t* new_len, void* ws,
                       void* stream);

/*
 * skipkv_select_fill_red -- skipkv_select_fill with the token-level redundancy of Section 4.1 ("Token Redundancy
 * Score" paragraph, as computed by skipkv_token_redundancy) deciding inside the cut sentence: its tokens leave in
 * increasing order of sigma * tok_imp[t] - (1 - sigma) * tok_red[t], Eq. "I_final" per token (the penalty is the same
 * for all tokens of a sentence and does not change their order).  The key is formed in fp32, every operation rounded
 * to nearest; equal keys: the earlier token stays first.  tok_red: device fp32, one value per cache row with the row
 * indexing of K (read only).  Everything else as skipkv_select_fill.
 */
int skipkv_select_fill_red(const skipkv_shape* shape, const skipkv_params* params, const float* sent_score,
                           const float* tok_imp, const float* tok_red, const int32_t* sent_off,
                           const int32_t* n_sent, uint8_t* keep, uint8_t* tok_keep, int32_t* kept_idx,
                           int32_t* n_kept, int32_t* new_len, void* ws, void* stream);
int skipkv_compact_fill(const skipkv_shape* shape, void* K, void* V, const uint8_t* keep,
                        const uint8_t* tok_keep, int32_t* sent_off, int32_t* sent_id, int32_t* n_sent,
                        int32_t* kv_len, int32_t* index_map, void* ws, void* stream);

/*
 * skipkv_token_redundancy -- the token-redundancy equation of Section 4.1 at token granularity: per slab
 * with N = kv_len[b][h] live rows,
 *   Kbar_t = K_t / (|K_t|_2 + eps),   G = Kbar Kbar^T  (N x N),
 *   tok_red[i] = (1/N) sum_{j != i} exp(G_ji) / sum_{k != j} exp(G_jk)
 * (row softmax with the diagonal excluded, then the column mean; the values of a slab sum to 1; N = 1 gives
 * 0).  This is what skipkv_score computes over pooled sentence keys, taken over the slab's own key rows:
 * the cost grows with N^2, so it is meant for caches near the budget (N about B + the decode interval).
 * K: device bf16 cache (read only).  tok_red: device fp32, one value per cache row with the row indexing of
 * K; rows at and beyond kv_len are not written.  params->eps is used; shape->total_rows must be the exact
 * row count of K.  Launch behaviour as skipkv_score.
 */
int skipkv_token_redundancy(const skipkv_shape* shape, const skipkv_params* params, const void* K,
                            const int32_t* kv_len, float* tok_red, void* ws, void* stream);

/*
 * skipkv_append_step -- the whole pre-eviction update of Algorithm 1 for one decode step (range append of
 * Eq. "before" included), on the device.  Per (b, h): the new K/V row is written at kv_len and kv_len is
 * incremented (as skipkv_append); the range list follows: when new_sent[b] != 0 (the previous token closed a
 * sentence) or the slab has no sentence yet, a new sentence starts at this token with
 * sent_id = gen_id[b]; the last sentence then ends at the newest token (sent_off[n_sent] = kv_len, entries
 * above it mirror the length).  If q_win is non-null the step's query q[b][*] replaces slot `slot`
 * (0 <= slot < window, host value, normally step % window) of the observation window q_win[b][*][slot].
 * new_sent: device u8 [batch].  gen_id: device int32 [batch].  q: device bf16 [batch][Hq][128].
 * A full slab (kv_len == cap) is left unchanged, a full range list (n_sent == max_sent) lets the token join
 * the last sentence; both raise SKIPKV_STATUS_BAD_TABLE.
 */
int skipkv_append_step(const skipkv_shape* shape, void* K, void* V, const void* k_new, const void* v_new,
                       int32_t* kv_len, int32_t* sent_off, int32_t* sent_id, int32_t* n_sent,
                       const uint8_t* new_sent, const int32_t* gen_id, void* q_win, const void* q,
                       int32_t slot, void* ws, void* stream);

/*
 * skipkv_decode_attn_paged -- skipkv_decode_attn over a paged cache, the layout of a paged-attention server
 * (the paper's second host, appendix "System-Level Evaluation on vLLM").  K_pages and V_pages are pools of pages
 * of SKIPKV_PAGE_ROWS rows of 128 bf16 (32 KB per page and tensor, page p at byte offset p * 32768, 16-byte
 * aligned base); token t of slab (b, h) lives in row t % SKIPKV_PAGE_ROWS of page
 * block_table[b][h][t / SKIPKV_PAGE_ROWS].  block_table: device int32 [batch][Hk][max_pages] (entries beyond the
 * live pages are not read).  kv_len[b][h] <= min(cap[b], max_pages * SKIPKV_PAGE_ROWS); shape->slab_off is not
 * used.  Everything else as skipkv_decode_attn; the two give bit-identical results for the same rows.
 */
#define SKIPKV_PAGE_ROWS 128
int skipkv_decode_attn_paged(const skipkv_shape* shape, const void* q, const void* K_pages, const void* V_pages,
                             const int32_t* block_table, int32_t max_pages, const int32_t* kv_len, void* out,
                             void* hidden, const void* steer_vec, const float* alpha, const uint8_t* flag,
                             void* ws, void* stream);

/*
 * skipkv_score_paged -- skipkv_score over the paged cache of skipkv_decode_attn_paged (same pool, block table and
 * page size).  Only K is read.  tok_imp (nullable) is laid out per slab with a stride of max_pages *
 * SKIPKV_PAGE_ROWS floats: tok_imp[(b*Hk + h) * max_pages * SKIPKV_PAGE_ROWS + t].  Requires
 * max_pages * SKIPKV_PAGE_ROWS <= max_cap + SKIPKV_PAGE_ROWS - 1 (the workspace is sized from max_cap) and
 * shape->total_rows = rows of the pool.  shape->slab_off is not used.  Every other argument and every output as
 * skipkv_score; the two give bit-identical results for the same rows.
 */
int skipkv_score_paged(const skipkv_shape* shape, const skipkv_params* params, const void* K_pages,
                       const int32_t* block_table, int32_t max_pages, const void* q_win, const int32_t* kv_len,
                       const int32_t* sent_off, const int32_t* n_sent, float* tok_imp, float* sent_imp,
                       float* sent_red, float* sent_lam, float* sent_score, void* ws, void* stream);

/*
 * skipkv_compact_paged -- skipkv_compact over the paged cache: the surviving rows of slab (b, h) are packed to the
 * front of the slab's own pages, in the order of its block table (row t of the packed slab is row
 * t % SKIPKV_PAGE_ROWS of page block_table[b][h][t / SKIPKV_PAGE_ROWS]); the block table itself is not changed, so
 * the pages behind the new kv_len are free for the caller to return to its pool.  Two slabs must not share a
 * page.  index_map (nullable) has a stride of max_pages * SKIPKV_PAGE_ROWS per slab, like tok_imp of
 * skipkv_score_paged.  Everything else, and the resulting rows, tables and lengths, as skipkv_compact.
 */
int skipkv_compact_paged(const skipkv_shape* shape, void* K_pages, void* V_pages, const int32_t* block_table,
                         int32_t max_pages, const uint8_t* keep, int32_t* sent_off, int32_t* sent_id,
                         int32_t* n_sent, int32_t* kv_len, int32_t* index_map, void* ws, void* stream);

/*
 * skipkv_decode_step -- one decode step of Algorithm 2 for one layer in a single launch: skipkv_append_step
 * followed by skipkv_decode_attn (attention over the cache including the new row, steering add), fused.
 * The new K/V row of (b, h) is written at kv_len_in[b][h] and attended to; the range list and the observation
 * window are updated as by skipkv_append_step (q_win nullable: window untouched).  Lengths are read from
 * kv_len_in and the new lengths written to kv_len_out, which must be a different buffer (the caller swaps the
 * two between steps); sent_off, sent_id and n_sent are updated in place.  A slab without room is left
 * unchanged (kv_len_out = kv_len_in, attention over the old rows) and raises SKIPKV_STATUS_BAD_TABLE, as does a
 * full range list.  Contiguous slabs only.  Other arguments as skipkv_decode_attn.
 */
int skipkv_decode_step(const skipkv_shape* shape, const void* q, const void* k_new, const void* v_new, void* K,
                       void* V, const int32_t* kv_len_in, int32_t* kv_len_out, int32_t* sent_off,
                       int32_t* sent_id, int32_t* n_sent, const uint8_t* new_sent, const int32_t* gen_id,
                       void* q_win, int32_t slot, void* out, void* hidden, const void* steer_vec,
                       const float* alpha, const uint8_t* flag, void* ws, void* stream);

/*
 * skipkv_decode_step_paged -- skipkv_decode_step over the paged cache: the new row of (b, h) goes to row
 * kv_len_in % SKIPKV_PAGE_ROWS of page block_table[b][h][kv_len_in / SKIPKV_PAGE_ROWS], which the caller must have
 * assigned before the call (a slab needs (kv_len_in + 1) rows' worth of pages; room is
 * min(cap[b], max_pages * SKIPKV_PAGE_ROWS)).  Everything else as skipkv_decode_step.
 */
int skipkv_decode_step_paged(const skipkv_shape* shape, const void* q, const void* k_new, const void* v_new,
                             void* K_pages, void* V_pages, const int32_t* block_table, int32_t max_pages,
                             const int32_t* kv_len_in, int32_t* kv_len_out, int32_t* sent_off, int32_t* sent_id,
                             int32_t* n_sent, const uint8_t* new_sent, const int32_t* gen_id, void* q_win,
                             int32_t slot, void* out, void* hidden, const void* steer_vec, const float* alpha,
                             const uint8_t* flag, void* ws, void* stream);

/*
 * skipkv_decode_attn_static -- skipkv_decode_attn for callers that cannot allocate device
 * memory and so have no workspace to pass.  (The paper has no counterpart: this is a packaging
 * variant of the same operation, not another step of the method.)  Typical callers: a serving
 * process whose start-up gave all free HBM to the KV-cache pool, so that any later cudaMalloc
 * fails; or an extension that must not call cudaMalloc because that call synchronises the whole
 * device and stalls the process's other streams.  The kernel's scratch (partial results and
 * arrival counters) lives in a fixed array inside the library instead, about 2 MB, which each
 * GPU that loads the library holds until the process exits.  This function calls no cudaMalloc,
 * cudaFree or other allocating routine.
 *
 * Arguments as skipkv_decode_attn, except that there is no workspace and that `status` (device,
 * one uint32, nullable, caller-owned) receives the SKIPKV_STATUS_* bits by bitwise OR; the caller
 * clears it.  Limits: batch * n_kv_heads <= SKIPKV_STATIC_MAX_SLABS, otherwise
 * SKIPKV_ERR_UNSUPPORTED is returned, nothing is enqueued, and skipkv_last_cuda_error() says
 * which limit was exceeded.
 *
 * The first call on a device looks up the array's device address (with that device current);
 * make that first call before any stream capture begins.  Every call
 * on a device shares the one array: each call first clears the counters it needs at zero (on
 * `stream`), and two calls whose GPU work overlaps (different streams, or different threads
 * without ordering between them) race on it and give undefined results.  Calls that follow one
 * another on one stream are safe.
 */
#define SKIPKV_STATIC_MAX_SLABS 256
int skipkv_decode_attn_static(const skipkv_shape* shape, const void* q, const void* K, const void* V,
                              const int32_t* kv_len, void* out, void* hidden, const void* steer_vec,
                              const float* alpha, const uint8_t* flag, uint32_t* status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SKIPKV_H_ */
