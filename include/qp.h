/*
 * qp.h — C ABI of the quantized-pruning KV-cache library for NVIDIA B200 (sm_100a).
 *
 * The library implements the data-parallel hot path of "quantized pruning"
 * (arXiv 2412.12706, Sec. 3 "Methods", paragraph "Quantized Pruning"): at the end
 * of prefill each layer's KV cache is pruned to a fixed number of tokens per KV
 * head and the kept keys/values are quantized; every decode step then attends
 * over the dequantized packed cache.
 *
 * Conventions for every call
 *   - "device" pointers are CUDA device memory of the current device, "host"
 *     pointers ordinary host memory.  The caller owns every buffer; the library
 *     never allocates, frees, synchronises or copies to the host.  All work is
 *     enqueued on `stream` (a cudaStream_t passed as void*; NULL = default stream)
 *     and buffers must stay alive until the stream has passed that point.
 *   - bf16 / fp16 tensors are raw 16-bit patterns, row-major and contiguous, base
 *     addresses 16-byte aligned.  Inputs must be finite.  Magnitudes: K, V and Q_win of the
 *     prefill-side calls up to 65504 (the fp16 range of the stored scale and zero).  The decode
 *     calls multiply in fp16 on the tensor cores (query x key scale, softmax weight x value scale)
 *     and need   max|q| * max|K| <= 2^19   and   max|V| <= 4096   over the tensors of a call, K and V
 *     being the values that were quantized into the cache (at 16 bit: max|q| <= 65504 only).
 *     Beyond that a product may overflow fp16 and the output holds inf or NaN; nothing checks it.
 *   - Host-checkable errors are returned before anything is launched and leave
 *     the outputs untouched.  Launch failures are reported as QP_ERR_CUDA from
 *     cudaGetLastError() without synchronising.
 *   - Results are deterministic: same inputs, same bits.
 *
 * Notation (the paper's where it has one): Bt batch, Hq query heads, Hkv KV heads,
 * G = Hq/Hkv, D head dimension, L prompt length, w observation window,
 * P = L - w, B = bits in {2,4,8,16}, g = quantization group size,
 * n = n_keep = tokens kept per KV head (the w window tokens included).
 */
#ifndef QP_H_
#define QP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  QP_OK = 0,
  QP_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, Hq % Hkv != 0, w >= L, even pool ... */
  QP_ERR_UNSUPPORTED = 2, /* bits not in {2,4,8,16}, group not in {32,64,128}, D not in {64,128}, G > 8, w > 64, pool > 65,
                             batch * n_kv_heads * L >= 2^31 - 128 in the score stage */
  QP_ERR_BUDGET = 3,      /* budget gives n <= w, n is not a whole number of groups, or no room to append */
  QP_ERR_WORKSPACE = 4,   /* workspace too small */
  QP_ERR_ALIGNMENT = 5,   /* a base pointer is not 16-byte aligned */
  QP_ERR_CUDA = 6         /* a launch failed */
} qp_status;

#define QP_MAX_LAYERS 128

/*
 * Packed pruned cache of one layer: a plain descriptor (host memory) of
 * caller-allocated device buffers.  It may be copied freely; the library keeps no
 * reference to it.  Layout of the buffers (wpg = g*B/32 words per group):
 *
 *   k_codes  uint32 [Bt, Hkv, n/g, D, wpg]   key groups: one channel, g consecutive KEPT tokens
 *   k_scale  fp16   [Bt, Hkv, n/g, D]        (per-channel quantization, KIVI; Sec. 2 and 5.3)
 *   k_zero   fp16   [Bt, Hkv, n/g, D]
 *   v_codes  uint32 [Bt, Hkv, n, D/g, wpg]   value groups: one kept token, g consecutive channels
 *   v_scale  fp16   [Bt, Hkv, n, D/g]        (per-token quantization)
 *   v_zero   fp16   [Bt, Hkv, n, D/g]
 *
 * Element e of a group sits in word e / (32/B) at bit offset (e mod (32/B)) * B.
 * A stored value is reconstructed as code * scale + zero (Eq. 5).
 * B = 16: k_codes / v_codes hold the gathered bf16 rows [Bt, Hkv, n, D] and the four
 * scale/zero pointers are unused (sizes 0).
 * Kept tokens are stored in ascending order of their position in the prompt.
 *
 * Room for tokens appended during decoding (Eq. 2): n_cap > n_keep sizes every array for n_cap
 * tokens per KV head (read n_cap for n in the shapes above: the stride from one (batch, KV head)
 * to the next is that of n_cap tokens), of which the first n_keep are in use.  n_cap = 0 means
 * n_cap = n_keep (no room).  For B < 16 n_cap is a multiple of g.
 */
typedef struct qp_cache {
  int32_t batch, n_q_heads, n_kv_heads, head_dim, bits, group, n_keep, n_cap;
  size_t k_codes_bytes, v_codes_bytes;
  size_t k_meta_bytes; /* bytes of k_scale; k_zero has the same size */
  size_t v_meta_bytes; /* bytes of v_scale; v_zero has the same size */
  void *k_codes, *v_codes, *k_scale, *k_zero, *v_scale, *v_zero; /* device */
} qp_cache;

/* Text for a status code (static storage, never NULL). */
const char* qp_status_string(qp_status s);

/*
 * Token budget (Appendix B "Memory Budgets"; Fig. 2: tokens x bits is held
 * constant).  budget_bits is the token-bit product per (KV head, channel), e.g.
 * 512 tokens at 16 bit = 8192.  *n_keep = min(budget_bits / bits, L); scale/zero
 * metadata is not counted.  QP_ERR_BUDGET if n_keep <= w or (bits < 16 and n_keep
 * is not a multiple of group).  Host only.
 */
qp_status qp_n_keep(int64_t budget_bits, int bits, int group, int L, int w, int32_t* n_keep /* host, out */);

/*
 * Fills the shape fields and the four byte sizes of *out for the layout above and
 * sets the six pointers to NULL.  Host only.
 */
qp_status qp_cache_layout(int batch, int n_q_heads, int n_kv_heads, int head_dim, int bits, int group,
                          int n_keep, qp_cache* out /* host, out */);

/* The same with room for n_cap >= n_keep tokens per KV head (see qp_cache). */
qp_status qp_cache_layout_cap(int batch, int n_q_heads, int n_kv_heads, int head_dim, int bits, int group,
                              int n_keep, int n_cap, qp_cache* out /* host, out */);

/* Bytes of device scratch that qp_compress_layer / qp_window_scores need (0 on invalid shapes). */
size_t qp_compress_workspace_bytes(int batch, int n_q_heads, int n_kv_heads, int head_dim, int L, int w);

/* Bytes of device scratch that qp_decode_attn needs for this cache (0 on an invalid descriptor).
 * For qp_decode_attn_layers pass the sum over the layers. */
size_t qp_decode_workspace_bytes(const qp_cache* cache /* host */);

/*
 * S1, observation-window scores.  The paper names its pruning method (SnapKV,
 * Sec. 4 "Setup", Appendix B: the last 32 tokens are always retained) without
 * defining it; this is the rule implemented.  For each KV head and each of its G
 * query heads h and window rows i (position p = P + i):
 *   S[j] = q[h,i].k[j] / sqrt(D) for j <= p;  Pr = softmax_j(S)
 *   vote[j] = sum_h sum_i Pr_{h,i}[j]                          j < P
 *   scores[j] = (sum_{|t| <= (pool-1)/2} vote[j+t], zero outside [0,P)) / pool
 * Q_win bf16 [Bt,Hq,w,D], K bf16 [Bt,Hkv,L,D] (device) -> scores fp32 [Bt,Hkv,P] (device).
 * pool must be odd (1 = no pooling) and at most 65.
 * Error word: the score sweeps wait on hardware barriers (copies into shared memory, tensor-core
 * completion) with a bounded number of polls.  A block whose wait runs out stops, and the 32-bit
 * word at byte offset qp_compress_workspace_bytes(...) - 256 of the workspace becomes 1; the
 * scores (and everything qp_compress_layer derives from them) are then invalid.  The word is
 * cleared at the start of every qp_window_scores / qp_compress_layer(s) call (stream-ordered) and
 * can be read by the caller once the stream has passed the call.  It is 0 in every correct run.
 */
qp_status qp_window_scores(const void* Q_win, const void* K, int batch, int n_q_heads, int n_kv_heads,
                           int head_dim, int L, int w, int pool, float* scores, void* workspace,
                           size_t workspace_bytes, void* stream);

/*
 * S2, per-head top-k (Sec. 3 "KV Pruning": keep s < n tokens).  Of the P prefix
 * positions of each (batch, KV head) the n_keep - w with the largest score are
 * kept, equal scores resolved toward the lower position; the w window positions
 * P..L-1 are always kept.  scores fp32 [Bt,Hkv,P] (device, no NaN) ->
 * kept_idx int32 [Bt,Hkv,n_keep] (device), ascending.
 */
qp_status qp_select_topk(const float* scores, int batch, int n_kv_heads, int L, int w, int n_keep,
                         int32_t* kept_idx, void* stream);

/*
 * S3, gather + quantize + pack (Eq. 4: Q(G) = round((G - z)/s), s = (m - z)/(2^B - 1),
 * z = min, m = max of the group).  Stored precision: z is rounded down and s rounded
 * up to fp16, and the codes are computed in fp32 from the STORED z and s as
 * clamp(rint((x - z)/s), 0, 2^B - 1) (true division, ties to even); s = 0 gives codes 0.
 * K, V bf16 [Bt,Hkv,L,D], kept_idx int32 [Bt,Hkv,n_keep] ascending, each < L (device).
 * cache: shape fields as from qp_cache_layout, pointers set by the caller.
 */
qp_status qp_gather_quantize(const void* K, const void* V, const int32_t* kept_idx, int L,
                             const qp_cache* cache /* host */, void* stream);

/*
 * Prefill-side path of one layer: S1 -> S2 -> S3 ("Quantized Pruning": prune first,
 * then quantize the preserved states).  n_keep follows qp_n_keep(budget_bits, bits,
 * group, L, w); cache->n_keep etc. must agree with it (QP_ERR_BUDGET otherwise).
 * Outputs: the cache buffers and kept_idx int32 [Bt,Hkv,n_keep] (device).
 */
qp_status qp_compress_layer(const void* K, const void* V, const void* Q_win, int batch, int n_q_heads,
                            int n_kv_heads, int head_dim, int L, int w, int64_t budget_bits, int bits,
                            int group, int pool, const qp_cache* cache /* host */,
                            int32_t* kept_idx /* device */, void* workspace, size_t workspace_bytes,
                            void* stream);

/*
 * The same prefill-side path for n_layers independent layers of one shape (1 <= n_layers <=
 * QP_MAX_LAYERS, batch * n_layers * n_kv_heads <= 65535) with one launch per stage instead of one per
 * stage and layer: a layer of a short prompt leaves most of the GPU idle, several at once do not
 * (layers of different sequences at the same depth, or a measurement over synthetic layers).
 * K, V, Q_win, kept_idx are HOST arrays of device pointers, budget_bits a HOST array (budgets and so
 * n_keep may differ per layer), caches a HOST array; shapes, bits, group and pool are shared.
 * workspace: qp_compress_workspace_bytes(batch * n_layers, ...) bytes.  Results are identical, bit for
 * bit, to n_layers calls of qp_compress_layer.
 */
qp_status qp_compress_layers(int n_layers, const void* const* K, const void* const* V, const void* const* Q_win,
                             int batch, int n_q_heads, int n_kv_heads, int head_dim, int L, int w,
                             const int64_t* budget_bits /* host */, int bits, int group, int pool,
                             const qp_cache* caches /* host */, int32_t* const* kept_idx, void* workspace,
                             size_t workspace_bytes, void* stream);

/*
 * S4 + S5, decode-step attention over the packed cache (Eq. 3 on the dequantized
 * cache of Eq. 5): out[b,h,:] = softmax_t(q[b,h].K'[t] / sqrt(D)) V' over the n kept
 * tokens of KV head h / G, no mask.  q, out bf16 [Bt,Hq,D] (device).  The token
 * range is split across workers and the partial results merged; workspace (device,
 * 16-byte aligned, contents irrelevant) holds the partials.  Calls run in stream order
 * unless qp_decode_overlap has been enabled for the stream (below).  Calls on different
 * streams must not share a workspace.
 */
qp_status qp_decode_attn(const void* q, const qp_cache* cache /* host */, void* out, void* workspace,
                         size_t workspace_bytes, void* stream);

/*
 * Lets consecutive decode calls on `stream` overlap on the GPU (enable != 0) or returns the stream
 * to plain stream order (0, the default).  No counterpart in the paper: a launch-level measure.
 * Enabled, a decode call's attention kernel is launched so that it may begin while the previous
 * decode call's merge step still runs, which hides the launch gap and the merge step between the
 * calls of a decode loop.  The library keeps this safe against its own calls: it starts a call early
 * only if the call reads none of the previous decode call's out buffers (q and the cache arrays are
 * checked against them), alternates between two halves of the workspace (calls of different sizes
 * may share one workspace: where their halves would meet, the later call simply waits), and falls
 * back to stream order after any of its calls that writes a cache.  Its kernels guarantee that at
 * most two consecutive decode calls are in flight at a time.  Results are as if the calls ran one
 * after the other.
 * What the caller promises while it is enabled: whatever ELSE is enqueued on the stream between two
 * decode calls (kernels or copies that are not calls of this library) writes nothing that the later
 * call reads (its q, its cache arrays).  A loop that computes each layer's q just before attending
 * with it must leave the setting off.  Host call, takes effect from the next decode call on the
 * stream; the setting is per (device, stream) and is forgotten, falling back to the default, if more
 * than 256 streams are in use.
 */
qp_status qp_decode_overlap(void* stream, int enable);

/*
 * The same decode attention for n_layers independent layers in one pair of
 * launches (1 <= n_layers <= QP_MAX_LAYERS).  q, caches, out are HOST arrays of
 * length n_layers; q[l], out[l] are device pointers.  All caches must agree in
 * batch, heads and head_dim; n_keep may differ per layer.  bits and group may differ too
 * (the per-layer token/precision mixes of Sec. 5.4: some layers at 4 bit with 4x the tokens,
 * others at 8 or 16 bit): layers of equal (bits, group) then share a launch pair and the
 * classes run one after the other, results as for separate calls.
 */
qp_status qp_decode_attn_layers(int n_layers, const void* const* q, const qp_cache* caches,
                                void* const* out, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Tokens appended during decoding that have not been quantized yet (host descriptor, caller-
 * allocated device buffers).  Eq. 2 appends the new token's key and value to the cache; the paper
 * does not say how a quantized cache takes single tokens in, and a key group spans g tokens, so:
 * appended tokens wait in bf16 in this tail (fewer than g per KV head), attention runs over the
 * packed tokens followed by the tail, and when the tail holds g tokens they are quantized by
 * Eq. 4 exactly like g kept tokens of the prompt and become tokens n_keep .. n_keep+g-1 of the
 * packed cache.  B = 16 needs no tail (rows go straight into the cache); the pointers may be NULL.
 */
typedef struct qp_tail {
  int32_t n_tail;         /* tokens in the tail, 0 <= n_tail < group; maintained by qp_append_kv */
  int32_t reserved_;
  void *k_tail, *v_tail;  /* device bf16 [Bt, Hkv, group, D] each, 16-byte aligned */
} qp_tail;

/*
 * Eq. 2 for one decode step: appends the key/value rows of the new token, k_new, v_new bf16
 * [Bt,Hkv,D] (device), to each of n_layers caches (1 <= n_layers <= QP_MAX_LAYERS; k_new, v_new
 * HOST arrays of device pointers; caches, tails HOST arrays, updated in place).
 * B < 16: the rows are written to tail slot n_tail; if that fills the tail, its g tokens are
 * quantized into key group n_keep/g and value rows n_keep.. of the cache (same arithmetic as
 * qp_gather_quantize), n_keep grows by g and n_tail returns to 0.  B = 16: the rows are written
 * to token n_keep of the cache and n_keep grows by 1.  One or two launches for all layers; the
 * layers need not agree in n_keep or n_tail but must agree in shape, bits and group.
 * QP_ERR_BUDGET, before anything is launched or changed, when a cache has no room left
 * (n_keep + g > n_cap for a flush, n_keep + 1 > n_cap at 16 bit).
 */
qp_status qp_append_kv_layers(int n_layers, const void* const* k_new, const void* const* v_new,
                              qp_cache* caches /* host, in/out */, qp_tail* tails /* host, in/out */,
                              void* stream);
/* The same for one layer. */
qp_status qp_append_kv(const void* k_new, const void* v_new, qp_cache* cache /* host, in/out */,
                       qp_tail* tail /* host, in/out */, void* stream);

/*
 * Decode attention (Eq. 3) over the packed tokens followed by the tail's tokens: the softmax runs
 * over n_keep + n_tail tokens.  Arguments as for qp_decode_attn_layers / qp_decode_attn plus the
 * tails (HOST array; tails[l].n_tail may be 0, tails may be NULL for "no tail anywhere").
 * The tail is read in full precision by the merge step.
 */
qp_status qp_decode_attn_tail_layers(int n_layers, const void* const* q, const qp_cache* caches,
                                     const qp_tail* tails, void* const* out, void* workspace,
                                     size_t workspace_bytes, void* stream);
qp_status qp_decode_attn_tail(const void* q, const qp_cache* cache /* host */, const qp_tail* tail /* host */,
                              void* out, void* workspace, size_t workspace_bytes, void* stream);

/*
 * The other quantization strategies of the paper's ablation (Sec. 5.3 "Quantization methods"; Appendix B
 * "KV quantization").  The method's own arrangement is KIVI's (keys per channel, values per token, no
 * filtering); the ablation also runs
 *   - the FlexGen arrangement: keys AND values quantized token by token, g consecutive channels of one
 *     token per group (k_axis = 1; the paper's FlexGen runs use g = 64), and
 *   - outlier filtering for either arrangement: numbers with |x| > outlier_threshold (6 in the paper,
 *     about 1 % of the cache) are left out of their group's min/max, get code 0, and are kept in 16 bit in
 *     a side list; reconstruction takes the listed value instead of code * scale + zero.  A group that
 *     consists of outliers only has scale = zero = 0.
 * With k_axis = 1 the key arrays of qp_cache have the value arrays' shapes: k_codes [Bt,Hkv,n,D/g,wpg],
 * k_scale, k_zero [Bt,Hkv,n,D/g] (same byte sizes as before).
 * Side list of one tensor (device arrays, caller-allocated): for every (batch, KV head) the outliers in
 * ascending order of t*D + d (t = index among the kept tokens, d = channel):
 *   idx int32 [Bt,Hkv,cap], val bf16 [Bt,Hkv,cap], cnt int32 [Bt,Hkv] (-1: more than cap outliers, list invalid),
 *   tile_ptr int32 [Bt,Hkv,ceil(n/32)+1]: the entries of tokens 32i..32i+31 are [tile_ptr[i], tile_ptr[i+1]).
 * outlier_threshold <= 0 or +inf: no filtering (the side lists are ignored and may be zeroed structs).
 */
typedef struct qp_side {
  int32_t cap, reserved_;
  int32_t* idx;
  void* val;
  int32_t* cnt;
  int32_t* tile_ptr;
} qp_side;
typedef struct qp_strategy {
  int32_t k_axis;            /* 0: keys per channel (KIVI); 1: keys per token (FlexGen) */
  float outlier_threshold;   /* <= 0 or inf: off */
  qp_side k_side, v_side;
} qp_strategy;

/* S3 under a strategy: as qp_gather_quantize (bits < 16), plus the side lists when filtering is on. */
qp_status qp_gather_quantize_ex(const void* K, const void* V, const int32_t* kept_idx, int L,
                                const qp_cache* cache /* host */, const qp_strategy* strategy /* host */,
                                void* stream);
/* S4 + S5 under a strategy: as qp_decode_attn for a cache written by qp_gather_quantize_ex with the same
 * strategy.  Runs in plain stream order.  workspace: qp_decode_workspace_bytes(cache) bytes. */
qp_status qp_decode_attn_ex(const void* q, const qp_cache* cache /* host */, const qp_strategy* strategy /* host */,
                            void* out, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Head-level token budgets: the KV heads of a layer share the layer's budget and keep different numbers of
 * tokens.  The paper runs two pruning methods of this kind (Ada-KV, HeadKV: Related Work "KV Pruning", Sec. 4
 * "Setup", Table 1) and says of them only that they retain different tokens per head; the rule here: within a
 * batch entry the Hkv * (n_mean - w) prefix positions with the largest scores over all KV heads are marked
 * (equal scores: lower head, then lower position); a head's share is its marked positions plus its w window
 * tokens, rounded down to whole units of `unit` tokens, at least the smallest unit count above w, at most L
 * rounded down to units; if raising small heads pushed the total above Hkv * n_mean, the largest heads (lowest
 * first among equals) give back one unit at a time.
 * scores fp32 [Bt,Hkv,P] (device, from qp_window_scores) -> n_keep_heads int32 [Bt,Hkv] (device).  The caller
 * copies the counts to the host to size one cache per (batch, KV head) (descriptors with batch = 1,
 * n_kv_heads = 1, n_q_heads = G) and then runs qp_select_topk / qp_gather_quantize(_ex) per head on that
 * head's slice of scores, K and V, and qp_decode_attn_layers(_ex) over the heads' descriptors.  With
 * unit = group the heads' caches satisfy the per-channel key grouping of the main path; the paper pairs
 * these methods with the per-token arrangement (k_axis = 1).
 * workspace: qp_head_budgets_workspace_bytes(...) bytes, 16-byte aligned.  unit >= 1, n_mean > w.
 */
size_t qp_head_budgets_workspace_bytes(int batch, int n_kv_heads, int L, int w, int n_mean);
qp_status qp_head_budgets(const float* scores, int batch, int n_kv_heads, int L, int w, int n_mean, int unit,
                          int32_t* n_keep_heads, void* workspace, size_t workspace_bytes, void* stream);

/* qp_decode_attn_ex for n_layers caches of one shape, bits and group in one launch pair (n_keep may differ: e.g. the
 * per-head caches of a head-level budget).  Side lists (filtering) are supported for n_layers = 1 only:
 * QP_ERR_UNSUPPORTED otherwise.  workspace: the sum of qp_decode_workspace_bytes over the caches. */
qp_status qp_decode_attn_layers_ex(int n_layers, const void* const* q, const qp_cache* caches /* host */,
                                   const qp_strategy* strategy /* host */, void* const* out, void* workspace,
                                   size_t workspace_bytes, void* stream);

/*
 * Debug build only (libqp_checked.so, compiled with -DQP_CHECKED; no counterpart in the paper).  In that build
 * every index a kernel reads from DEVICE memory and then uses as an address (the kept positions given to the
 * gather / quantize kernels, the side lists' tile pointers and entries), and every output position the top-k kernels
 * compute from their counts, is compared with its limit first; a
 * violation never traps: the first one is recorded, all are counted, and the access goes to element 0 or is
 * skipped.  This call synchronises the device, copies the record to words4 (host: 1 + site of the first
 * violation or 0, the offending index, its limit, the number of violations) and clears it.  Indices that
 * come from host fields (n_keep, n_cap, n_tail, shapes) are validated by every entry point before any launch in
 * both builds.  The normal build returns QP_ERR_UNSUPPORTED and zeros.
 */
qp_status qp_debug_check(uint32_t* words4 /* host, out */);

/*
 * Decode attention without any caller-supplied scratch.  (The paper has no counterpart to this
 * call; it exists for integration reasons only.)  Some hosts of this library cannot give it
 * scratch memory: a serving process that hands all device memory to its own arena at start-up,
 * so that a later cudaMalloc fails or is forbidden by policy; a latency-critical decode loop that
 * may not risk the device-wide synchronisation an allocation can cause; a plugin interface that
 * passes tensors in and out but offers no way to request temporaries.  For them the split
 * partials of qp_decode_attn live in an array of QP_STATIC_SCRATCH_BYTES that is part of the
 * library image: every GPU on which the library is loaded holds these bytes until the process
 * exits.
 *
 * Same computation and result as qp_decode_attn(q, cache, out, ...); q, out bf16 [Bt,Hq,D] device.
 * Returns QP_ERR_WORKSPACE, before launching anything, when this cache needs more scratch than
 * QP_STATIC_SCRATCH_BYTES (sum over batch x KV heads x token splits x G of (D+2) floats): use
 * qp_decode_attn with your own workspace then.  It calls no cudaMalloc/cudaFree and no allocating
 * library routine.  The first call on each device looks up the array's device address (with that
 * device current); make that first call outside any stream capture.  All calls on a device share
 * the one array and it keeps the previous call's contents (nothing in it needs clearing: each
 * call writes every record it later reads), so two calls on different streams race on it;
 * serialise them on one stream or with events.
 */
#define QP_STATIC_SCRATCH_BYTES (4u << 20)
qp_status qp_decode_attn_static(const void* q, const qp_cache* cache /* host */, void* out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* QP_H_ */
