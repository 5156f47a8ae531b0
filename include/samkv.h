/*
 * samkv.h — C ABI of the SamKV hot path for NVIDIA B200 (sm_100a).
 *
 * The library sparsifies a multiple-context KV cache (per-document K/V that were prefilled
 * independently of one another) and attends over what survives, following
 * "Sparse Attention across Multiple-context KV Cache" (SamKV):
 *
 *   samkv_score    pooled query, personalised query (Eq. 1), inner-product block scores (Sec. 3.2)
 *   samkv_select   protected initial/local blocks + per-context top-k of the middle (Sec. 3.2, 4.1)
 *   samkv_compact  gather of the kept K/V rows into one compact cache, original order (Sec. 3.2)
 *   samkv_update   write recomputed rows back: Overwrite or Fusion (Sec. 3.3, Eq. 4)
 *   samkv_attn     GQA attention of a prefill chunk / decode step over the compact cache (Sec. 3.3)
 *
 * Conventions
 *   - Every tensor pointer is a DEVICE pointer owned by the caller, innermost dimension
 *     contiguous, base address 16-byte aligned, unless the comment says "host".
 *     Arrays marked "host" are read during the call and may be freed right after it returns.
 *   - Calls validate their arguments on the host, then only enqueue kernels on `stream`
 *     (a cudaStream_t passed as void*; NULL = the default stream).  They do not allocate,
 *     free or synchronise (samkv_poll_status is the one call that synchronises).
 *   - Plain stream order holds for every argument: whatever earlier work on `stream` wrote (Q
 *     from a projection kernel, the cache from samkv_update, cache_len from the previous call)
 *     is seen by the call.  Some kernels are launched so that their set-up overlaps the tail of
 *     the kernel before them (programmatic dependent launch); they read nothing the caller
 *     passes before that kernel has completed.
 *   - A handle owns no memory: scratch lives in the caller's `workspace`.  Calls that use the
 *     same handle must be ordered on one stream (they share the workspace).
 *   - On a host-detected error a call returns a non-zero status and launches nothing.
 *     Nothing traps or aborts.  There is no CPU fallback.
 *   - Shapes: L layers, Bt batch elements (independent requests that share the context
 *     lengths), Hq query heads, Hkv KV heads (Hq % Hkv == 0, G = Hq/Hkv), d = head_dim in {64,128},
 *     D contexts with ctx_offsets[c] .. ctx_offsets[c+1] on the concatenated token axis of
 *     length L_tot, B = block_size (selection unit, power of two <= 64; 1 = single tokens),
 *     units are counted from each context's own start (the last one may be short),
 *     nb_c = ceil(L_c / B), U_tot = sum nb_c.
 *   - Protected units of a context: every unit that overlaps its first n_init or last n_local
 *     tokens (n_init, n_local multiples of B).  If some L_c is not a multiple of B, n_local
 *     must be >= B so that the short tail unit is protected and every head keeps the same
 *     number of tokens.
 */
#ifndef SAMKV_H_
#define SAMKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SAMKV_MAX_CTX 128        /* most contexts per request */
#define SAMKV_MAX_UNITS_PER_CTX 49152  /* most selection units in one context */

typedef struct samkv_ctx* samkv_handle_t; /* opaque */

typedef enum {
  SAMKV_OK = 0,
  SAMKV_ERR_INVALID_ARG = 1,  /* null / misaligned pointer, inconsistent sizes */
  SAMKV_ERR_UNSUPPORTED = 2,  /* head_dim, dtype, block_size or size outside what is built */
  SAMKV_ERR_WORKSPACE = 3,    /* workspace smaller than samkv_workspace_bytes() */
  SAMKV_ERR_CAPACITY = 4,     /* compact cache capacity too small */
  SAMKV_ERR_BUDGET = 5,       /* k_units[c] outside [protected units, nb_c] */
  SAMKV_ERR_CUDA = 6,         /* a CUDA runtime call failed (launch error, wrong device) */
  SAMKV_ERR_DEVICE_CHECK = 7  /* a kernel recorded a failed device-side check */
} samkv_status_t;

typedef enum { SAMKV_F32 = 0, SAMKV_BF16 = 1 } samkv_dtype_t;
typedef enum { SAMKV_UPDATE_OVERWRITE = 0, SAMKV_UPDATE_FUSION = 1 } samkv_update_mode_t;

/* Problem shape shared by all calls. */
typedef struct {
  int32_t n_layers, batch, n_q_heads, n_kv_heads, head_dim;
  int32_t n_ctx;               /* D, 1 .. SAMKV_MAX_CTX */
  const int32_t* ctx_offsets;  /* host [n_ctx+1], ascending, ctx_offsets[0] == 0 */
  int32_t block_size;          /* B; the paper runs with 64 */
  int32_t n_init, n_local;     /* protected tokens per context; the paper runs with 64 and 128 */
  int32_t dtype;               /* samkv_dtype_t of K, V, Q, Qloc, Knew, Vnew, Kc, Vc, O */
} samkv_shape_t;

/* ---- handle, workspace, status -------------------------------------------------------- */

/* Bytes of device scratch the calls below need for this shape: the personalised query
 * vectors of samkv_score and the split-KV partial results of samkv_attn with up to
 * max_q_tokens query tokens over a cache of cache_capacity slots.  Returns 0 on a bad shape. */
size_t samkv_workspace_bytes(const samkv_shape_t* shape, int32_t max_q_tokens, int32_t cache_capacity);

/* Creates a handle bound to CUDA device `device` and to `workspace` (device pointer, 256-byte
 * aligned, workspace_bytes long, caller-owned, must outlive the handle).  Queries device
 * properties and enqueues one small memset on the default stream; allocates no device memory. */
samkv_status_t samkv_create(samkv_handle_t* out, int device, void* workspace, size_t workspace_bytes);
samkv_status_t samkv_destroy(samkv_handle_t h);
/* Host-side switch of a handle (no GPU work, takes effect with the next samkv_attn call on the handle).
 * on != 0: the caller keeps copy-like kernels (samkv_compact, samkv_update of other layers) running on another
 * stream while attention is in flight.  samkv_attn then uses, for bf16 prefill chunks with d = 128 and at least
 * 128 packed rows, a kernel that is slower on its own but leaves registers and shared memory on every SM for those
 * kernels' CTAs; the default kernel fills its SMs.  Results obey the same bounds either way.  The paper has no
 * counterpart: this is scheduling advice (Sec. 3.3 only fixes what attention computes). */
samkv_status_t samkv_attn_share_sm(samkv_handle_t h, int32_t on);

/* Synchronises `stream`, then returns SAMKV_ERR_DEVICE_CHECK if any kernel since the last poll
 * recorded a failed device-side check (and clears the record), SAMKV_ERR_CUDA if the stream
 * reports an error, else SAMKV_OK. */
samkv_status_t samkv_poll_status(samkv_handle_t h, void* stream);
const char* samkv_status_string(samkv_status_t s);

/* ---- host-side helpers (no GPU work) --------------------------------------------------- */

/* Units kept per context under a sequence budget given in basis points (1500 = 15 %, the
 * sequence ratio the paper reports in Table 1): k_c = clamp(floor(budget_bp * nb_c / 10000),
 * protected units of c, nb_c).  k_units_out: host [n_ctx]. */
samkv_status_t samkv_budget_units(const samkv_shape_t* shape, int32_t budget_bp, int32_t* k_units_out);

/* Number of protected units per context (host [n_ctx], may be NULL) and, for a given k_units
 * (host [n_ctx], may be NULL), the number of tokens S the compact cache will hold. */
samkv_status_t samkv_layout(const samkv_shape_t* shape, const int32_t* k_units, int32_t* n_protected_out,
                            int32_t* total_units_out, int32_t* kept_tokens_out);

/* ---- the five steps --------------------------------------------------------------------- */

/* Scoring (Sec. 3.1 mean pooling; Eq. 1; Sec. 3.2 inner products with block-mean keys).
 *   K     [L, Bt, Hkv, L_tot, d]
 *   Q     [L, Bt, T_q, Hq, d]          the user query's Q rows of each layer
 *   Qloc  [L, Bt, D, T_loc, Hq, d]     each document's local-position Q cache (T_loc = 1 accepts a
 *                                      pre-pooled vector); NULL or use_bias == 0 => Q^ = Q_que
 * Per (layer, batch, query head): Q_que = mean_t Q, q_loc_j = mean_t Qloc_j,
 *   Q^_i = Q_que + 1/(D-1) * sum_{j != i} |cos(Q_que, q_loc_j)| * q_loc_j   (weight 0 for a zero norm;
 *   D == 1 => Q^ = Q_que), folded to KV heads by the mean over the G query heads of a group.
 * Per (layer, batch, KV head, token t of context i): s = <q_i, K_t> in fp32 (no scaling);
 * unit score = mean of s over the unit's real tokens (== <q_i, mean K> by linearity).
 *   scores_out fp32 [L, Bt, Hkv, U_tot]
 *   qhat_out   fp32 [L, Bt, D, Hkv, d], optional (NULL: kept in the workspace only) */
samkv_status_t samkv_score(samkv_handle_t h, const samkv_shape_t* shape, const void* K, const void* Q, int32_t T_q,
                           const void* Qloc, int32_t T_loc, int32_t use_bias, float* scores_out, float* qhat_out,
                           void* stream);

/* Selection (Sec. 3.2: initial and local positions are kept in full, the middle is sparsified;
 * here under a fixed per-context budget).  Per (layer, batch, KV head, context c): keep the
 * protected units plus the k_units[c] - n_protected_c middle units with the largest score;
 * of equal scores the lower index wins (-0 and +0 compare equal).
 *   scores   fp32 [L, Bt, Hkv, U_tot]
 *   k_units  host [n_ctx], units kept per context, protected ones included
 *   sel_out  int32 [L, Bt, Hkv, S_u], S_u = sum k_units: global unit ids, ascending;
 *            context c's segment starts at sum_{c'<c} k_units[c'] */
samkv_status_t samkv_select(samkv_handle_t h, const samkv_shape_t* shape, const float* scores, const int32_t* k_units,
                            int32_t* sel_out, void* stream);

/* Compaction (Sec. 3.2: initial + selected + local rows joined in their original order).
 *   Kc[l,b,h,slot,:] = K[l,b,h,tok(slot),:], same for V; slots run over (context, token) ascending.
 *   K, V      [L, Bt, Hkv, L_tot, d].  Either may also be a pointer into PINNED HOST memory that the
 *             device can address (cudaHostAlloc / cudaHostRegister under unified addressing): the kernel
 *             then pulls just the kept rows across the bus, so only the kept share is ever loaded to the GPU
 *             (the paper's "sequence ratio", Table 1).  V can always stay on the host; K can when the scores
 *             came from the block representatives (samkv_score_blocks), since token-mode samkv_score reads
 *             all of K on the device anyway
 *   sel       int32 [L, Bt, Hkv, S_u] as written by samkv_select; k_units host [n_ctx]
 *   Kc, Vc    [L, Bt, Hkv, cache_capacity, d]; slots >= S are left untouched
 *   cache_len int32 [L, Bt], set to S (the number of kept tokens)
 *   inv_map   int32 [L, Bt, Hkv, L_tot], optional: slot of each token, -1 where this head did not
 *             keep it (the paper's "blank" position when layers/heads are aligned for recomputation)
 * Returns SAMKV_ERR_CAPACITY if cache_capacity < S.  Copies are bit-exact. */
samkv_status_t samkv_compact(samkv_handle_t h, const samkv_shape_t* shape, const void* K, const void* V,
                             const int32_t* sel, const int32_t* k_units, void* Kc, void* Vc, int32_t cache_capacity,
                             int32_t* cache_len, int32_t* inv_map, void* stream);

/* Selection and compaction in one launch (Sec. 3.2: score -> select -> initial + selected + local rows joined in
 * their original order).  Same results, bit for bit, as samkv_select followed by samkv_compact: sel_out, Kc, Vc,
 * cache_len and inv_map are written exactly as those two calls write them; one CTA selects the units of one
 * (layer, batch, KV head, context) and gathers their rows right away.  Arguments and errors as for the two calls
 * (K and V may be pinned host memory). */
samkv_status_t samkv_select_compact(samkv_handle_t h, const samkv_shape_t* shape, const float* scores,
                                    const int32_t* k_units, const void* K, const void* V, int32_t* sel_out, void* Kc,
                                    void* Vc, int32_t cache_capacity, int32_t* cache_len, int32_t* inv_map, void* stream);

/* The whole sparsification in one call: samkv_score, then samkv_select_compact.  scores_out and sel_out are outputs
 * like those of the separate calls (and must be given: the steps hand their data over through them).  Every argument
 * is validated before anything is enqueued. */
samkv_status_t samkv_sparsify(samkv_handle_t h, const samkv_shape_t* shape, const void* K, const void* V, const void* Q,
                              int32_t T_q, const void* Qloc, int32_t T_loc, int32_t use_bias, const int32_t* k_units,
                              float* scores_out, int32_t* sel_out, void* Kc, void* Vc, int32_t cache_capacity,
                              int32_t* cache_len, int32_t* inv_map, void* stream);

/* Composite cache of the protected positions only (Sec. 3.1 "Generate generic query vector": the initial and
 * local K/V of all contexts, concatenated; also the "no-selection" ablation of Sec. 4.1).  Same result as
 * samkv_select with k_units = protected units followed by samkv_compact, without scores or a unit list: the
 * kept rows are two contiguous ranges per context.  The user query is then prefilled over it with samkv_attn
 * (Kq/Vq appended), and the pooled Q of that pass is the Q_que that samkv_score takes.
 * Arguments as for samkv_compact; cache_len is set to the protected token count (samkv_layout's kept tokens
 * for k_units = protected units). */
samkv_status_t samkv_compact_protected(samkv_handle_t h, const samkv_shape_t* shape, const void* K, const void* V,
                                       void* Kc, void* Vc, int32_t cache_capacity, int32_t* cache_len,
                                       int32_t* inv_map, void* stream);

/* Write-back of recomputed rows (Sec. 3.3).  For every recomputed token r and every KV head that
 * kept it (slot = inv_map[l,b,h,tok_ids[l,r]] >= 0):
 *   overwrite: Kc[slot] = Knew[r], Vc[slot] = Vnew[r]
 *   fusion (Eq. 4): theta = cos(new, old) over the d elements of the row (1 if a norm is zero),
 *                   row = theta*new + (1-theta)*old in fp32, rounded to nearest-even in dtype;
 *                   K rows and V rows each use their own theta.
 *   tok_ids    int32 [L, R] global token ids on the concatenated axis, -1 = skip; ids of one layer
 *              must be distinct
 *   Knew, Vnew [L, Bt, R, Hkv, d] */
samkv_status_t samkv_update(samkv_handle_t h, const samkv_shape_t* shape, void* Kc, void* Vc, int32_t cache_capacity,
                            const int32_t* inv_map, const int32_t* tok_ids, int32_t R, const void* Knew,
                            const void* Vnew, int32_t mode, void* stream);

/* Attention of a query chunk over the compact cache of one layer (Sec. 3.3: the incremental
 * prefill of the user query over the new sparse cache, and the decode steps after it).
 *   Kc, Vc    [L, Bt, Hkv, cache_capacity, d]; `layer` picks the slab
 *   cache_len int32 [L, Bt] (device).  Slots < cache_len[layer,b] are visible to every query token.
 *   Q         [Bt, T_q, Hq, d] fresh query rows of this step
 *   Kq, Vq    [Bt, T_q, Hkv, d] optional (both or neither): the chunk's own keys/values, written to
 *             slots cache_len .. cache_len+T_q-1 and attended causally (token t sees appended slots <= t);
 *             afterwards cache_len[layer,b] += T_q.  The caller guarantees cache_len + T_q <= cache_capacity
 *             (a violation is recorded as a device check and the append is skipped).
 *   scale     softmax scale; <= 0 selects 1/sqrt(d)
 *   O         [Bt, T_q, Hq, d] = softmax(scale * Q Kc^T + mask) Vc, query head hq reads KV head hq/G
 *   lse       fp32 [Bt, Hq, T_q] optional: log of the softmax denominator
 * bf16 inputs: products on tensor cores with fp32 accumulation, probabilities rounded to bf16
 * before the PV product.  fp32 inputs: fp32 FMA throughout. */
samkv_status_t samkv_attn(samkv_handle_t h, const samkv_shape_t* shape, int32_t layer, void* Kc, void* Vc,
                          int32_t cache_capacity, int32_t* cache_len, const void* Q, int32_t T_q, const void* Kq,
                          const void* Vq, float scale, void* O, float* lse, void* stream);

/* The same attention for n consecutive layers, layer0 .. layer0 + n - 1, in one call: for callers that hold the
 * queries of several layers at once (the data-parallel setting in which samkv_score .. samkv_update also take all
 * layers per call).  One grid then covers every (layer, batch, KV head, row tile), which keeps all SMs busy where a
 * single layer has fewer tiles than the GPU has SMs and leaves no gap between layers.
 *   Kc, Vc, cache_len   as for samkv_attn (the whole [L, ...] tensors; the call offsets them to layer0)
 *   Q, O                [n, Bt, T_q, Hq, d];  Kq, Vq [n, Bt, T_q, Hkv, d] optional;  lse [n, Bt, Hq, T_q] optional
 * The workspace must be sized for the n * Bt requests of the call: samkv_workspace_bytes with a shape whose batch is
 * n * Bt (SAMKV_ERR_WORKSPACE otherwise).  Per layer the result obeys the bounds of samkv_attn; the number of KV
 * splits, and with it the rounding order, may differ from a per-layer call. */
samkv_status_t samkv_attn_layers(samkv_handle_t h, const samkv_shape_t* shape, int32_t layer0, int32_t n, void* Kc,
                                 void* Vc, int32_t cache_capacity, int32_t* cache_len, const void* Q, int32_t T_q,
                                 const void* Kq, const void* Vq, float scale, void* O, float* lse, void* stream);

/* ---- the paper's dynamic selection: Top-P per document, then Top-K across documents --------------- */

#define SAMKV_MAX_STAR_LAYERS 64

/* Dynamic Top-P (Sec. 3.2, Eq. 2; consolidated over the stable layers N*, Eq. 3).  Per stable layer n, batch
 * element, KV head and document i:
 *   s_anc = score of the anchor = token-weighted mean of the protected (initial + local) units' scores
 *   s_max, s_min = scores of the document's max / min blocks (max_units / min_units: device int32 [L, Bt, D],
 *                  global unit ids from the offline attention analysis of App. A.1), or, when the pointer is
 *                  NULL, the largest / smallest middle-unit score
 *   P^(n) = (s_max - s_anc) / (s_max - s_min)  if s_anc in (s_min, s_max],  else 0      (also 0 without middle units)
 * P_out[b, i] = mean over n in N* and over the KV heads (the paper has no head index).
 *   scores      fp32 [L, Bt, Hkv, U_tot] from samkv_score
 *   star_layers host [n_star], 1 <= n_star <= SAMKV_MAX_STAR_LAYERS, layer indices in [0, L)
 *   P_out       device fp32 [Bt, D] */
samkv_status_t samkv_topp(samkv_handle_t h, const samkv_shape_t* shape, const float* scores, const int32_t* star_layers,
                          int32_t n_star, const int32_t* max_units, const int32_t* min_units, float* P_out,
                          void* stream);

/* Host helper: from one request's ratios P (host [D]) the number of middle units retrieved per document,
 * cand[i] = floor(P[i] * middle units of i), the cross-context K = floor(sum cand / D), the length
 * S_u = protected units + K of every selection list, and the kept-token count S.  Outputs may be NULL. */
samkv_status_t samkv_topp_plan(const samkv_shape_t* shape, const float* P, int32_t* cand_out, int32_t* K_out,
                               int32_t* S_u_out, int32_t* kept_tokens_out);

/* Cross-context Top-K (Sec. 3.2, last paragraph).  Per (layer, batch, KV head): document i retrieves its cand[i]
 * best middle units (ties: lower index); their scores are min-max normalised inside the document over its
 * middle units ((u - min) / (max - min), 0 if max == min); the K = floor(sum cand / D) best of all retrieved
 * units are kept (equal normalised scores: lower global unit id), together with every protected unit.
 *   cand       host [D]
 *   scratch    device, 16-byte aligned, at least samkv_select_cross_scratch_bytes(shape, cand) bytes, owned by
 *              the caller and free again when the call's work on `stream` has finished; it holds one
 *              (key, unit id) pair per retrieved unit.  With cand == NULL the size helper returns the bound
 *              for any cand (every middle unit retrieved).
 *   sel_out    int32 [L, Bt, Hkv, S_u] ascending global unit ids, S_u = protected units + K
 *   counts_out int32 [L, Bt, Hkv, D] optional: units kept per document (they differ from head to head)
 * SAMKV_ERR_BUDGET if some cand[i] exceeds the document's middle units; SAMKV_ERR_WORKSPACE if scratch is short. */
size_t samkv_select_cross_scratch_bytes(const samkv_shape_t* shape, const int32_t* cand);
samkv_status_t samkv_select_cross(samkv_handle_t h, const samkv_shape_t* shape, const float* scores,
                                  const int32_t* cand, void* scratch, size_t scratch_bytes, int32_t* sel_out,
                                  int32_t* counts_out, void* stream);

/* Compaction for a selection list whose split between documents is free (as samkv_select_cross writes it):
 * sel int32 [L, Bt, Hkv, S_u] ascending global unit ids that contain every short tail unit.  Otherwise as
 * samkv_compact (V may be pinned host memory; cache_len set to the kept-token count; optional inv_map). */
samkv_status_t samkv_compact_units(samkv_handle_t h, const samkv_shape_t* shape, const void* K, const void* V,
                                   const int32_t* sel, int32_t S_u, void* Kc, void* Vc, int32_t cache_capacity,
                                   int32_t* cache_len, int32_t* inv_map, void* stream);

/* Number of kernels one samkv_attn call with these sizes launches on the device of `h` (append of the chunk when
 * `appended`, the attention kernel, the merge of KV splits where the attention kernel does not merge them itself).
 * For launch accounting; returns 0 for arguments samkv_attn would refuse. */
int32_t samkv_attn_kernel_count(samkv_handle_t h, const samkv_shape_t* shape, int32_t T_q, int32_t cache_capacity,
                                int32_t appended);

/* ---- block representatives (Sec. 3.2: a block's representative is the mean of its tokens' keys) ------------ */

/* Kbar[l,b,h,u,:] = mean over the tokens of unit u of K[l,b,h,t,:] (fp32 sum in a fixed order, one rounding to the
 * storage dtype; a short tail unit averages the tokens it has).  Query-independent: run once per stored document.
 *   K    [L, Bt, Hkv, L_tot, d]      Kbar [L, Bt, Hkv, U_tot, d], same dtype, 16-byte aligned */
samkv_status_t samkv_block_means(samkv_handle_t h, const samkv_shape_t* shape, const void* K, void* Kbar, void* stream);

/* samkv_score on the representatives: scores[l,b,h,u] = <q^_c, Kbar[l,b,h,u,:]> for u in context c, which equals
 * the block-mean of the token scores up to the one rounding of Kbar (inner products are linear).  Reads d*e bytes
 * per unit instead of per token.  Other arguments, outputs and errors as for samkv_score; `shape` is the token-level
 * shape (block_size = B), the same one samkv_select / samkv_compact take afterwards. */
samkv_status_t samkv_score_blocks(samkv_handle_t h, const samkv_shape_t* shape, const void* Kbar, const void* Q,
                                  int32_t T_q, const void* Qloc, int32_t T_loc, int32_t use_bias, float* scores_out,
                                  float* qhat_out, void* stream);

/* ---- cross-layer alignment of the sparse caches (Sec. 3.3 "Recomputation") ------------------------ */

#define SAMKV_FLAG_KEPT 1       /* some KV head of the layer keeps the token (not a blank position) */
#define SAMKV_FLAG_RECOMPUTE 2  /* K/V of the token are recomputed at this layer (rule 2) */
#define SAMKV_FLAG_OUTPUT 4     /* the layer must produce the token's output: a higher layer recomputes it (rule 1) */
#define SAMKV_FLAG_PAD_REUSE 8  /* blank here but on the forward path: the token's prefilled K/V entry is used */

/* Pad -> merge -> recompute plan.  Layers (and heads) keep different tokens; laying every layer over the union
 * of all layers' kept tokens aligns them, with blanks where a layer keeps nothing.  Per (layer n, batch b, token t):
 *   KEPT       inv_map[n,b,h,t] >= 0 for some head h
 *   RECOMPUTE  t is in tok_ids[n] and KEPT (a listed token that is blank at layer n has no entry to refresh)
 *   OUTPUT     RECOMPUTE holds for t at some layer m > n (its K/V there need the outputs of all layers below)
 *   PAD_REUSE  OUTPUT and not RECOMPUTE and not KEPT
 *   inv_map     int32 [L, Bt, Hkv, L_tot] as written by samkv_compact / samkv_compact_units
 *   tok_ids     int32 [L, R] (device) recompute lists as for samkv_update, -1 = unused entry; R may be 0
 *   flags_out   uint8 [L, Bt, L_tot]
 *   merged_ids  int32 [Bt, L_tot]: the merged axis, ascending token ids kept by any layer, then -1
 *   merged_len  int32 [Bt]
 *   run_ids     int32 [L, Bt, run_capacity]: ascending tokens with RECOMPUTE or OUTPUT (the layer's forward pass),
 *               then -1; run_len int32 [L, Bt] always holds the full count
 * A list longer than run_capacity is truncated and recorded as a device check (samkv_poll_status); so is a token
 * id >= L_tot.  The caller removes the padding again by writing results through inv_map (samkv_update). */
samkv_status_t samkv_align(samkv_handle_t h, const samkv_shape_t* shape, const int32_t* inv_map, const int32_t* tok_ids,
                           int32_t R, uint8_t* flags_out, int32_t* merged_ids, int32_t* merged_len, int32_t* run_ids,
                           int32_t run_capacity, int32_t* run_len, void* stream);

/* ---- scoring without any allocation ------------------------------------------------------ */

/* (No counterpart in the paper: this entry point exists for deployment reasons only.)
 * Same result as samkv_score, for callers that cannot call cudaMalloc or hand over a workspace:
 * a serving engine whose memory pool already owns all of HBM, or a latency-critical section in
 * which an allocation (which may synchronise the whole device) is not allowed.  It takes no handle.
 * The personalised query vectors, the only scratch this step needs, live in a fixed array inside
 * the library's device image: SAMKV_STATIC_SCORE_MAX_FLOATS fp32 values (1 MiB), held by every GPU
 * that loads the library until the process exits.
 *   - n_layers * batch * n_ctx * n_kv_heads * head_dim must not exceed SAMKV_STATIC_SCORE_MAX_FLOATS
 *     (one layer of any configuration in this repository fits; call it layer by layer), otherwise
 *     SAMKV_ERR_WORKSPACE is returned and nothing is launched.
 *   - The first call on a device looks up the array's device address (once per device, with that
 *     device current).  Make that first call outside any stream capture.
 *   - All calls share the one array: two calls whose kernels can overlap on the GPU (different
 *     streams, or several threads) race on it.  Order them on one stream.  The array keeps the last
 *     call's contents; every element a call reads is rewritten by that call first, so no clearing
 *     is needed.
 *   - Calls no cudaMalloc / cudaFree or any other allocating routine.
 *   - There is no handle and therefore no status word: a device-side check that samkv_score would record for
 *     samkv_poll_status (a bounded wait inside the scoring kernel that ran out) is NOT reported by this entry
 *     point.  The kernel still gives up and returns, part of scores_out is then left unwritten, and the call
 *     has long returned SAMKV_OK.  A caller that needs that report uses samkv_score with a workspace.
 * Arguments as in samkv_score (K, Q, Qloc, scores_out are caller-owned device pointers). */
#define SAMKV_STATIC_SCORE_MAX_FLOATS (256 * 1024)
samkv_status_t samkv_score_static(const samkv_shape_t* shape, const void* K, const void* Q, int32_t T_q,
                                  const void* Qloc, int32_t T_loc, int32_t use_bias, float* scores_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SAMKV_H_ */
