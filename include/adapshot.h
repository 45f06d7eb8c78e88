/*
 * adapshot.h - C ABI of the B200 (sm_100a) AdapShot KV-reuse hot path.
 *
 * The path (paper Sec. 4): rank the cached shots for a query and take the top k
 * (Sec. 4.1/4.2), concatenate the selected shots' cached K/V in relevance order
 * and move K to its new contiguous positions by one more rotary rotation
 * (Sec. 4.3, Eq. 6-7), attend from the probe tokens to each probe's prefix of
 * that cache (Eq. 1 and the tree mask of Sec. 4.1), and take the entropy of the
 * probe's next-token distribution with the threshold rule (Eq. 2).
 *
 * Conventions shared by every call
 *  - Every function returns 0 (ADAPSHOT_OK) or a negative ADAPSHOT_E* code.
 *    Host-side argument checks happen before any launch; on error nothing is
 *    enqueued.  Nothing aborts, traps or throws.
 *  - Structs and `probe_nshots` are HOST memory, read during the call only.
 *    Every other pointer is a DEVICE pointer owned by the caller, 16-byte
 *    aligned, valid until the enqueued work has finished.  The library
 *    allocates no device memory; scratch comes from the caller's `ws`
 *    (size from the matching *_workspace_bytes function, 256-byte aligned).
 *  - Work is enqueued asynchronously on `stream` (a cudaStream_t passed as
 *    void*; NULL = the legacy default stream).  Calls are thread-compatible.
 *  - `status` is a device int32 the caller zeroes once; kernels only ever
 *    store a non-zero ADAPSHOT_E* code into it (capacity overflow, bad shot
 *    id, a pipeline wait that ran out).  The offending unit of work is
 *    skipped; no out-of-bounds access is made.  Read it after synchronising.
 *  - Layout names: B queries, k selected shots, P nested probes, T_q probe
 *    tokens, Hq / Hkv query / KV heads, G = Hq / Hkv, d = head_dim,
 *    nl = layer_end - layer_begin layers handled by one call.
 */
#ifndef ADAPSHOT_H_
#define ADAPSHOT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define ADAPSHOT_API __attribute__((visibility("default")))
#else
#define ADAPSHOT_API
#endif

#define ADAPSHOT_OK            0
#define ADAPSHOT_EINVAL       -1   /* null pointer, non-positive size, bad flag    */
#define ADAPSHOT_ESHAPE       -2   /* head_dim, head ratio, probe list, k > N ...  */
#define ADAPSHOT_EALIGN       -3   /* pointer not 16-byte aligned                  */
#define ADAPSHOT_ECAPACITY    -4   /* ctx_cap / workspace / static scratch too small */
#define ADAPSHOT_EUNSUPPORTED -5   /* dtype / mode this build has no kernel for    */
#define ADAPSHOT_ECUDA        -6   /* a CUDA runtime or driver call failed         */
#define ADAPSHOT_EINDEX       -7   /* device saw a shot id outside 0..n_shots-1    */
#define ADAPSHOT_ETIMEOUT     -8   /* device pipeline wait exceeded its limit      */

#define ADAPSHOT_F32   0
#define ADAPSHOT_BF16  1

/* Model shape (Sec. 4.2: L layers, H heads; grouped-query mapping h -> h / G). */
typedef struct adapshot_model {
  int32_t n_layers;       /* layers held by the pool                              */
  int32_t n_q_heads;      /* Hq                                                   */
  int32_t n_kv_heads;     /* Hkv, divides Hq                                      */
  int32_t head_dim;       /* d: 64 or 128                                         */
  int32_t dtype;          /* storage of pool / ctx / q / out: ADAPSHOT_F32 | BF16 */
  int32_t k_pos_mode;     /* 0: pool K carries no position (angle (o+t) theta);
                             1: pool K was rotated at its shot-local position t
                                (Sec. 4.3: prefilled alone from 0), angle o theta */
  double  rope_base;      /* theta_i = rope_base^(-2i/d)  (text after Eq. 6)      */
  float   softmax_scale;  /* 0 => 1/sqrt(d)  (Eq. 5 scaling)                      */
  int32_t reserved;
} adapshot_model_t;

/* Global cache pool (Sec. 4.2, Eq. 3), token-major so that one shot's block of
 * one layer is a single contiguous run:
 *   k, v : [n_layers][pool_tokens][Hkv][d]   (dtype of the model)
 *   shot i owns tokens shot_off[i] .. shot_off[i+1]-1 (lengths >= 1)
 *   emb  : fp32 [n_shots][emb_dim] shot embeddings for the relevance ranking   */
typedef struct adapshot_pool {
  int32_t        n_shots;
  int32_t        emb_dim;
  int64_t        pool_tokens;
  const int64_t* shot_off;   /* device, [n_shots + 1], ascending, shot_off[0] = 0 */
  const void*    k;          /* device */
  const void*    v;          /* device */
  const float*   emb;        /* device */
} adapshot_pool_t;

/* ---- Step 1: relevance ranking and top-k (Sec. 4.1 ranking; Sec. 4.2 "rank in
 * descending order and select the top k").  score[b][i] = cosine(q_emb[b],
 * emb[i]) with fp64 accumulation of the fp32 products (0 if either norm is 0);
 * sel_idx[b][r] = id of the r-th most relevant shot, equal scores ordered by
 * the lower id.  Nested probes use prefixes of sel_idx.
 *   q_emb [B][emb_dim] fp32; sel_idx [B][k] int32 out; sel_score [B][k] fp32 out
 *   or NULL.  Needs 1 <= k <= n_shots (else ADAPSHOT_ESHAPE); a pool of more than
 *   8192 shots (one sort chunk) takes k <= 4096 (else ADAPSHOT_EUNSUPPORTED: the
 *   chunks' candidate lists would not shrink from one merge round to the next).
 *   Scores are compared in fp64.                                                */
ADAPSHOT_API size_t adapshot_select_workspace_bytes(int32_t n_shots, int32_t B, int32_t k);
ADAPSHOT_API int adapshot_select(const adapshot_pool_t* pool, const float* q_emb, int32_t B, int32_t k,
                    int32_t* sel_idx, float* sel_score,
                    void* ws, size_t ws_bytes, int32_t* status, void* stream);

/* ---- Step 1 with the paper's own relevance score (Sec. 4.2, Eq. 5 and the ranking sentence
 * after it): attention of the query's Q at a representative layer against the cached K of every
 * shot.  Eq. 5 as printed normalises over one shot's own tokens (every shot's mean score is then
 * 1 / T_i, whatever the query); the reading taken is ONE softmax per query token and head over
 * the keys of the whole pool at that layer:
 *   a[t][h][j] = softmax_j( q[t][h] . k[layer][j][h / G] * scale ),  j over all pool tokens
 *   s[b][i]    = (1 / (T_q Hq)) sum_{t,h} sum_{j in shot i} a[t][h][j]      (sums to 1 over i)
 *   with ADAPSHOT_RELEVANCE_PER_TOKEN: s[b][i] / T_i (the mean score of one of its tokens).
 * Q and K enter as stored (no rotary rotation is applied here); scale = model->softmax_scale
 * or 1/sqrt(d).  sel_idx[b][r] = id of the r-th most relevant shot, equal scores by lower id.
 *   q [B][T_q][Hq][d] bf16; sel_idx [B][k] int32 out; sel_score [B][k] fp32 out or NULL.
 * bf16 tensor-core kernels (two passes over the layer's K: the normaliser, then the masses),
 * fp32 exponentials, fp64 accumulation of the masses (by atomics: the last bits of a score may
 * differ from run to run).  model->dtype must be ADAPSHOT_BF16; limits as adapshot_select,
 * pool_tokens < 2^31 - 256.                                                                 */
#define ADAPSHOT_RELEVANCE_PER_TOKEN 1u
ADAPSHOT_API size_t adapshot_select_attn_workspace_bytes(const adapshot_model_t* model, const adapshot_pool_t* pool,
                                            int32_t B, int32_t Tq, int32_t k);
ADAPSHOT_API int adapshot_select_attn(const adapshot_model_t* model, const adapshot_pool_t* pool, int32_t layer,
                         const void* q, int32_t B, int32_t Tq, int32_t k, uint32_t flags,
                         int32_t* sel_idx, float* sel_score, void* ws, size_t ws_bytes,
                         int32_t* status, void* stream);

/* ---- Step 2: KV-level concatenation with position re-encoding (Sec. 4.3,
 * Eq. 7; offsets follow the two-shot example: a shot placed after r others
 * starts at the sum of their lengths).
 *   ctx_off[b][r] = sum_{r'<r} T_{sel_idx[b][r']}, r = 0..k      (int64 out)
 *   v_ctx[b][l][o+t][h][:] = v_pool[layer_begin+l][shot_off[s]+t][h][:]  (bit copy)
 *   k_ctx[b][l][o+t][h][:] = Rot(k_pool[...], Delta theta), o = ctx_off[b][r],
 *   s = sel_idx[b][r], Delta = o+t (k_pos_mode 0) or o (k_pos_mode 1), with
 *   Rot(x)_i = x_i cos - x_{i+d/2} sin, Rot(x)_{i+d/2} = x_{i+d/2} cos + x_i sin
 *   (Eq. 6, half-split rotate_half).  Angles are formed in fp64, the rotation in
 *   fp32, bf16 results are rounded to nearest-even.
 *   k_ctx, v_ctx : [B][nl][ctx_cap][Hkv][d]; both NULL => only ctx_off is written
 *   (and, when ctx_cap > 0, the capacity is checked).
 *   Rows L .. min(roundup(L,128), ctx_cap)-1 of every (b, l) are zero-filled so
 *   that the attention kernel can read whole 128-token tiles.
 *   Device-detected: L > ctx_cap -> ADAPSHOT_ECAPACITY (tokens beyond the
 *   capacity are dropped); shot id out of range -> ADAPSHOT_EINDEX (the shot
 *   counts as length 0).  sel_idx need not come from adapshot_select.
 *   flags: 0, or ADAPSHOT_ASSEMBLE_KEEP_PLAN when ctx_off already holds the plan of
 *   the same sel_idx (an earlier call): it is then read, not written, so calls for
 *   further layer ranges may run on other streams while attention reads it.      */
#define ADAPSHOT_ASSEMBLE_KEEP_PLAN 1u
/*   ADAPSHOT_ASSEMBLE_K_ONLY: only k_ctx is written (v_ctx is ignored and may be NULL).  Eq. 7
 *   corrects the keys alone, so a consumer that reads V from the pool through the plan
 *   (adapshot_query_attn_vpool) needs no copy of it, and the gather moves half the bytes.    */
#define ADAPSHOT_ASSEMBLE_K_ONLY 2u
ADAPSHOT_API int adapshot_assemble_kv(const adapshot_model_t* model, const adapshot_pool_t* pool,
                         const int32_t* sel_idx, int32_t B, int32_t k,
                         int32_t layer_begin, int32_t layer_end,
                         void* k_ctx, void* v_ctx, int64_t ctx_cap,
                         int64_t* ctx_off, uint32_t flags,
                         int32_t* status, void* stream);

/* The same for the selected shots shot_begin .. k-1 only: positions from
 * ctx_off[b][shot_begin] on are written (and the zero fill after L), earlier positions
 * of k_ctx / v_ctx are left as they are.  Nested probes share their prefix (Sec. 4.1): a
 * cache assembled for the first shot_begin shots of the same sel_idx is extended in
 * place, at the cost of the new shots only.  0 <= shot_begin < k; ctx_off is written in
 * full (unless ADAPSHOT_ASSEMBLE_KEEP_PLAN).  shot_begin = 0 is adapshot_assemble_kv.   */
ADAPSHOT_API int adapshot_assemble_kv_from(const adapshot_model_t* model, const adapshot_pool_t* pool,
                              const int32_t* sel_idx, int32_t B, int32_t k, int32_t shot_begin,
                              int32_t layer_begin, int32_t layer_end,
                              void* k_ctx, void* v_ctx, int64_t ctx_cap,
                              int64_t* ctx_off, uint32_t flags,
                              int32_t* status, void* stream);

/* ---- Step 3: probe attention over the reused cache (Eq. 1; tree mask of
 * Sec. 4.1: probe j sees the first probe_nshots[j] shots, i.e. context tokens
 * 0 .. L_j-1 with L_j = ctx_off[b][probe_nshots[j]], and causally its own T_q
 * tokens, which sit at positions L_j .. L_j+T_q-1).  For row t and query head h
 * (KV head h / G): q' = Rot(q, (L_j+t) theta); keys = k_ctx[0..L_j) followed by
 * Rot(kq[t'], (L_j+t') theta), t' <= t; values = v_ctx[0..L_j) followed by
 * vq[t' <= t]; out = softmax(q' . keys * scale) . values.
 *   q   : [B][nl][P][T_q][Hq][d]   un-rotated   (bf16)
 *   kq,vq: [B][nl][P][T_q][Hkv][d] un-rotated   (bf16)
 *   out : [B][nl][P][T_q][Hq][d]   (bf16);  lse [B][nl][P][Hq][T_q] fp32 natural-log
 *         log-sum-exp of the scaled scores, or NULL
 *   probe_nshots : HOST int32 [P], strictly ascending, 1 <= n_j <= k
 *   k_ctx, v_ctx, ctx_cap, ctx_off: as written by adapshot_assemble_kv for the
 *   same B, k and layer range.
 * bf16 tensor-core kernel (tcgen05, fp32 accumulation, split over the context
 * with a log-sum-exp merge); model->dtype must be ADAPSHOT_BF16.
 * Limits of one call (ADAPSHOT_ESHAPE beyond them, nothing launched): P <= 16
 * probes, B * P <= 256 (probe, query) pairs, ctx_cap < 2^31 - 256.
 * Every wait inside the kernel is bounded by about two seconds of SM clock; a GPU
 * that is time-sliced with other work for longer than that in the middle of a
 * call can therefore report a spurious ADAPSHOT_ETIMEOUT in `status` (the
 * outputs of that call are then incomplete: repeat it).                         */
ADAPSHOT_API size_t adapshot_attn_workspace_bytes(const adapshot_model_t* model, int32_t B, int32_t P,
                                     int32_t Tq, int32_t n_layers_in_call, int64_t ctx_cap);
ADAPSHOT_API int adapshot_query_attn(const adapshot_model_t* model,
                        const void* k_ctx, const void* v_ctx, int64_t ctx_cap,
                        const int64_t* ctx_off, int32_t B, int32_t k,
                        const int32_t* probe_nshots, int32_t P,
                        const void* q, const void* kq, const void* vq, int32_t Tq,
                        int32_t layer_begin, int32_t layer_end,
                        void* out, float* lse, uint32_t flags,
                        void* ws, size_t ws_bytes, int32_t* status, void* stream);

/* ---- Steps 2 + 3 fused: the same attention, but the context K/V tiles are read from
 * the pool (through sel_idx / ctx_off) and K is re-encoded (Eq. 7) tile by tile in
 * shared memory on its way to the tensor cores, so that no assembled cache is written
 * to or read from HBM.  Results equal adapshot_assemble_kv + adapshot_query_attn up to
 * the rounding of the rotary table (fp32 (cos, sin) from fp64 angles, neighbouring rows
 * by one fp32 complex multiplication; K' rounded once to bf16 as in the materialised
 * path).  ctx_off: the plan written by adapshot_assemble_kv (plan-only call is enough)
 * for the same sel_idx; ctx_cap: an upper bound of every L (sizes the workspace: a row
 * maps of 2 * B * ctx_cap int32 and a table of ctx_cap * d * 4 bytes).  Both
 * k_pos_mode values are taken (1: every key of a shot is rotated by the angle of the
 * shot's first position, read from the same table).  Needs pool_tokens < 2^31.  Other
 * arguments as above.                                                                */
ADAPSHOT_API size_t adapshot_attn_fused_workspace_bytes(const adapshot_model_t* model, int32_t B, int32_t P,
                                           int32_t Tq, int32_t n_layers_in_call, int64_t ctx_cap);
ADAPSHOT_API int adapshot_query_attn_fused(const adapshot_model_t* model, const adapshot_pool_t* pool,
                              const int32_t* sel_idx, const int64_t* ctx_off, int64_t ctx_cap,
                              int32_t B, int32_t k, const int32_t* probe_nshots, int32_t P,
                              const void* q, const void* kq, const void* vq, int32_t Tq,
                              int32_t layer_begin, int32_t layer_end, void* out, float* lse,
                              uint32_t flags, void* ws, size_t ws_bytes, int32_t* status, void* stream);

/* ---- Step 3 over a cache that holds the re-encoded K only: the same attention, K tiles
 * from k_ctx (written by adapshot_assemble_kv with ADAPSHOT_ASSEMBLE_K_ONLY), V tiles copied
 * straight from the pool through sel_idx / ctx_off (Eq. 7 leaves V as it is, so its rows in
 * the pool are the rows of the assembled context).  Results equal adapshot_query_attn over
 * a full cache bit for bit in exact arithmetic (the same values reach the tensor cores; the
 * accumulation order is the same).  ctx_cap: the capacity k_ctx was assembled with (it also
 * sizes a row map of 2 * B * ctx_cap int32 in the workspace).  Needs pool_tokens < 2^31.
 * Other arguments, limits and error rules as adapshot_query_attn.                        */
ADAPSHOT_API size_t adapshot_attn_vpool_workspace_bytes(const adapshot_model_t* model, int32_t B, int32_t P,
                                           int32_t Tq, int32_t n_layers_in_call, int64_t ctx_cap);
ADAPSHOT_API int adapshot_query_attn_vpool(const adapshot_model_t* model, const adapshot_pool_t* pool,
                              const int32_t* sel_idx, const void* k_ctx, int64_t ctx_cap,
                              const int64_t* ctx_off, int32_t B, int32_t k,
                              const int32_t* probe_nshots, int32_t P,
                              const void* q, const void* kq, const void* vq, int32_t Tq,
                              int32_t layer_begin, int32_t layer_end, void* out, float* lse,
                              uint32_t flags, void* ws, size_t ws_bytes, int32_t* status, void* stream);

/* ---- Step 3 in the paper's literal form (Sec. 4.1, parallel multi-probe verification): ONE
 * sequence [shot_1 .. shot_n1, probe_1, shot_n1+1 .. shot_n2, probe_2, ...] with the tree mask
 * M_ij = 1 iff i is a token of probe_k and j belongs to its first n_k shots (plus, as causal
 * attention requires, the probe's own earlier tokens).  The sequence is described by a segment
 * table in HOST memory: seg_kind[i] is ADAPSHOT_SEG_SHOTS (seg_len[i] = number of selected
 * shots in the run, taken in sel_idx order) or ADAPSHOT_SEG_PROBE (seg_len[i] = tokens of the
 * probe).  Probes must each follow at least one new shot, have equal token counts, and the
 * sequence must end with a probe; at most 16 probes (ADAPSHOT_ESHAPE otherwise).  The shots'
 * K/V come from the assembled cache, so the tensors hold the probe tokens only, in sequence
 * order: q_seq [B][nl][N_probe_tokens][Hq][d], kq_seq / vq_seq [..][Hkv][d], out_seq like
 * q_seq.  No dense mask is materialised: a probe's row range of visible keys follows from the
 * table.  Position ids (shots keep 0 .. L-1 of their plain concatenation, token t of probe k
 * sits at L_k + t) are written to pos_seq [B][N_probe_tokens] int64 when it is not NULL.
 * adapshot_tree_layout is the table's parser alone (host only; probe_nshots [16] out).
 * Everything else as adapshot_query_attn.                                                  */
#define ADAPSHOT_SEG_SHOTS 0
#define ADAPSHOT_SEG_PROBE 1
ADAPSHOT_API int adapshot_tree_layout(const int32_t* seg_kind, const int32_t* seg_len, int32_t n_seg, int32_t k,
                         int32_t* probe_nshots, int32_t* P_out, int32_t* Tq_out);
ADAPSHOT_API int adapshot_tree_attn(const adapshot_model_t* model, const void* k_ctx, const void* v_ctx,
                       int64_t ctx_cap, const int64_t* ctx_off, int32_t B, int32_t k,
                       const int32_t* seg_kind, const int32_t* seg_len, int32_t n_seg,
                       const void* q_seq, const void* kq_seq, const void* vq_seq,
                       int32_t layer_begin, int32_t layer_end, void* out_seq, float* lse,
                       int64_t* pos_seq, uint32_t flags, void* ws, size_t ws_bytes, int32_t* status,
                       void* stream);

/* ---- Decoding over the chosen prefix (Sec. 4.1: the shot count that met the threshold is
 * "used for subsequent formal inference").  Query b continues over its first n_shots[b]
 * selected shots (context length L_b = ctx_off[b][n_shots[b]]) with T_own own tokens (its
 * query tokens and whatever has been generated so far) at positions L_b .. L_b + T_own - 1;
 * the call computes the rows of the LAST T_new of them (T_new = 1: one decode step; T_new =
 * T_own: the prefill of the query over the chosen prefix).  Row t sees the L_b context tokens
 * and the own tokens up to its own.
 *   n_shots : DEVICE int32 [B], 1 <= n_shots[b] <= k (e.g. derived from first_ok); a value
 *             outside that range is reported as ADAPSHOT_EINDEX in `status` and clamped
 *   q_new   : [B][nl][T_new][Hq][d];  k_own, v_own : [B][nl][T_own][Hkv][d]  (un-rotated)
 *   out     : [B][nl][T_new][Hq][d];  lse [B][nl][Hq][T_new] or NULL
 * Same kernels as adapshot_query_attn (a decode step is bound by the K/V bytes it reads, not
 * by the tensor cores); limits: B <= 256, T_own >= T_new >= 1.                              */
ADAPSHOT_API size_t adapshot_decode_workspace_bytes(const adapshot_model_t* model, int32_t B, int32_t T_new,
                                       int32_t T_own, int32_t n_layers_in_call);
ADAPSHOT_API int adapshot_decode_attn(const adapshot_model_t* model, const void* k_ctx, const void* v_ctx,
                         int64_t ctx_cap, const int64_t* ctx_off, int32_t B, int32_t k,
                         const int32_t* n_shots, const void* q_new, const void* k_own, const void* v_own,
                         int32_t T_new, int32_t T_own, int32_t layer_begin, int32_t layer_end,
                         void* out, float* lse, uint32_t flags, void* ws, size_t ws_bytes,
                         int32_t* status, void* stream);

/* ---- Step 4: confidence probe (Eq. 2 over the whole vocabulary, natural log)
 * and the threshold rule that follows it.
 *   H[r] = -sum_v p_v ln p_v, p = softmax(logits[r][0..V))          (fp32 out)
 *   first_ok[g] = smallest j in 0..rows_per_group-1 with
 *                 H[g*rows_per_group + j] <= tau, else -1   (int32 out, or NULL)
 *   logits [R][row_stride] fp32 or bf16 (dtype), row_stride in elements, rows
 *   16-byte aligned; one pass with a running maximum, fp32 accumulation.
 *   A logit at or below -2^97 (about -1.6e29) counts as -inf: it adds nothing; a row
 *   that holds nothing above it, and an all-NaN row, give H = 0.
 *   Limits: R a multiple of rows_per_group, rows_per_group <= 8192, and
 *   R * splits < 2^31, where splits <= 64 is the number of slices (multiples of 8192
 *   entries, one CTA each) a row is cut into; ADAPSHOT_ESHAPE otherwise.
 *   Ask adapshot_entropy_workspace_bytes for the scratch size (12 bytes per row and
 *   slice, rounded up to 256; it depends on R and V only, not on the device).     */
ADAPSHOT_API size_t adapshot_entropy_workspace_bytes(int32_t R, int32_t V);
ADAPSHOT_API int adapshot_entropy(const void* logits, int32_t dtype, int32_t R, int32_t V, int64_t row_stride,
                     float* H, float tau, int32_t rows_per_group, int32_t* first_ok,
                     void* ws, size_t ws_bytes, int32_t* status, void* stream);

/* ---- Step 4 over a token subset (Eq. 2 as printed: the entropy over the answer tokens
 * {Yes, No} of the probe prompt).  subset_ids: device int32 [n_subset] token ids.
 *   flags 0: p_v is taken from the softmax over the whole vocabulary and not renormalised,
 *            H = -sum_{v in S} p_v ln p_v  (at most n_subset / e; the case-study values the
 *            paper prints, two of which exceed ln 2, fit this reading of a two-token set);
 *   flags 1 (ADAPSHOT_ENTROPY_RENORM): q_v = p_v / sum_S p, H = -sum_S q_v ln q_v <= ln n_subset.
 * An id outside 0..V-1 is reported as ADAPSHOT_EINDEX in `status` and skipped.  Everything
 * else (threshold rule, layouts, workspace size) as adapshot_entropy.                      */
#define ADAPSHOT_ENTROPY_RENORM 1u
ADAPSHOT_API int adapshot_entropy_subset(const void* logits, int32_t dtype, int32_t R, int32_t V,
                            int64_t row_stride, const int32_t* subset_ids, int32_t n_subset, uint32_t flags,
                            float* H, float tau, int32_t rows_per_group, int32_t* first_ok,
                            void* ws, size_t ws_bytes, int32_t* status, void* stream);

/* ---- adapshot_entropy for callers that cannot provide or allocate scratch.
 * (No counterpart in the paper: this is a packaging variant of the call above.)
 * Meant for callers that must not call cudaMalloc, or hand out workspace, at the
 * point where they need the probe entropy: code living inside a serving process
 * whose device memory is fully owned by a pool allocator, plugins loaded into a
 * host that forbids allocation after start-up, and paths where an allocation's
 * implicit device synchronisation is not acceptable.  Same arguments, results
 * and error codes as adapshot_entropy, minus `ws`: the per-split states live in
 * a fixed 192 KiB device array inside the library (one per GPU that loads it,
 * held until the process exits).
 *  - Limit: R <= 16384 rows; more return ADAPSHOT_ECAPACITY and launch nothing.
 *    The rows are split as in adapshot_entropy, but never into more than
 *    floor(16384 / R) slices each (the array holds 16384 states).
 *  - The first call on each device looks up the array's device address (with
 *    that device current); make that first call outside any stream capture.
 *  - The call allocates and frees nothing, on the host or the device.
 *  - All calls share the one array, and it keeps whatever the last call left in
 *    it; every state a call reads is first written by that call, so stale
 *    contents are harmless, but two calls whose kernels overlap on the GPU
 *    (different streams, or different threads) race on it: serialise them.     */
ADAPSHOT_API int adapshot_entropy_static(const void* logits, int32_t dtype, int32_t R, int32_t V,
                            int64_t row_stride, float* H, float tau, int32_t rows_per_group,
                            int32_t* first_ok, int32_t* status, void* stream);

/* ---- Measurement aid (no counterpart in the paper).  adapshot_profile(1) makes every
 * later adapshot_query_attn / adapshot_query_attn_fused call record two CUDA events on the
 * caller's stream around its main (tensor-core) kernel; adapshot_profile_attn_main_ms()
 * waits for the last such call and returns that kernel's device time in milliseconds
 * (-1 if none).  Not thread-safe; leave it off (0) outside benchmarks and do not enable
 * it while a stream is being captured into a graph.                                   */
ADAPSHOT_API int adapshot_profile(int enable);
ADAPSHOT_API float adapshot_profile_attn_main_ms(void);

/* ---- Self-test of the failure path (no counterpart in the paper).  Every wait inside the
 * attention kernel is bounded: when a barrier is not completed within the limit the CTA
 * reports ADAPSHOT_ETIMEOUT in `status`, lets its copies land, frees its tensor memory and
 * returns.  This call runs that wait on a barrier nothing completes, with a limit of about
 * a millisecond: afterwards `status` holds ADAPSHOT_ETIMEOUT and cycles[0], cycles[1]
 * (device int64) the SM cycles the two waiting warps spent before giving up.  The kernel
 * ends normally; the context stays usable.                                               */
ADAPSHOT_API int adapshot_selftest_wait_timeout(int32_t* status, long long* cycles, void* stream);

ADAPSHOT_API const char* adapshot_strerror(int code);
ADAPSHOT_API int adapshot_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ADAPSHOT_H_ */
