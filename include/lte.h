/*
 * liblte — learnable-token-eviction (LTE) sparse attention for NVIDIA B200 (sm_100a).
 *
 * C ABI.  Every tensor pointer is a DEVICE pointer owned by the caller, contiguous with the
 * last index fastest and 16-byte aligned; `lte_shape` / `lte_conv` themselves are HOST structs
 * (their `w` / `bias` members are device pointers).  Unless a function says otherwise the
 * library allocates nothing and every call is asynchronous on `stream` (a cudaStream_t passed as
 * void*; NULL = the legacy default stream).  Scratch memory is the caller's: ask
 * lte_workspace_bytes() and pass at least that many bytes.
 *
 * State the library keeps between calls, all of it per device and none of it results: (1) on the
 * host, a small table per device ordinal, filled on first use under a mutex (SM count, the raised
 * dynamic-shared-memory limits of its kernels, one symbol address), so any number of host threads
 * may call into the library on any devices; (2) on each device, one status record per kernel
 * family (see lte_device_status) and the fixed scratch array of lte_attn_bwd_static.  Calls act
 * on the device that is current when they are made.
 *
 * Return value: LTE_OK (0) or a negative lte_status; nothing throws or aborts across the ABI.
 * Host-side validation happens before anything is launched.
 *
 * Notation (0-based positions): W = sliding window, i.e. query i sees keys i-W < j <= i
 * (W keys including itself); R = retain budget (the paper's b); sink = number of leading
 * positions that are always kept (the paper's s); K = taps of the scorer; half = K/2;
 * z = pre-sigmoid logit of the scorer, r = sigmoid(z) the retention score; a token is a
 * keep candidate iff r > tau, evaluated as z > logit(tau).
 */
#ifndef LTE_H_
#define LTE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum lte_status {
    LTE_OK = 0,
    LTE_ERR_INVALID_ARG = -1,      /* NULL pointer, misaligned pointer, non-positive size, even K, W < K ... */
    LTE_ERR_UNSUPPORTED = -2,      /* a shape or dtype no kernel covers (see each function)                 */
    LTE_ERR_WORKSPACE = -3,        /* ws_bytes smaller than lte_workspace_bytes() for this call             */
    LTE_ERR_CUDA = -4,             /* a CUDA runtime / driver call failed (launch, tensor-map encode ...)   */
    LTE_ERR_ARCH = -5,             /* current device is not compute capability 10.x                        */
    LTE_ERR_DEVICE_STATUS = -6     /* a kernel recorded an anomaly (bounded wait expired, bad state)        */
} lte_status;

enum { LTE_F32 = 0, LTE_BF16 = 1 };

typedef struct lte_shape {
    int32_t B, H, T, d;            /* batch, heads, sequence length, head dim (32, 64 or 128)            */
    int32_t W, R, sink;            /* window, retain budget, attention-sink size                          */
    float   tau;                   /* keep threshold on r; 0.5 in the paper.  tau <= 0 keeps every scored token */
    float   softmax_scale;         /* <= 0 selects 1/sqrt(d)                                               */
    int32_t dtype;                 /* LTE_F32 or LTE_BF16: storage type of q, k, v, o and their gradients   */
    int32_t group;                 /* grouped-query attention: query heads per key/value head; 0 or 1 = one.
                                      H counts key/value heads (k, v, z, idx, cnt, the cache); q, o, lse have
                                      H * group heads, those of one key/value head adjacent: [B, H, group, ...].
                                      dq has H * group heads too; dk, dv, dw, dbias are summed over a group          */
} lte_shape;

typedef struct lte_conv {
    int32_t n_layers;              /* 1: the single grouped conv layer 2d -> 1 per head; 3: the paper's stack (below) */
    int32_t kernel;                /* K taps, odd, centred (half past, self, half future)                   */
    int32_t dilation;              /* 1                                                                     */
    const float* w;                /* device, [H, K, 2d] fp32; channels [0,d) weigh k, [d,2d) weigh v       */
    const float* bias;             /* device, [H] fp32, or NULL for zero                                    */
} lte_conv;
/*
 * n_layers = 3 (d = 32 or 64; which calls take it is said below): the scorer of Section 3.1.1 with the hyper-parameters of
 * Appendix A: three grouped conv layers of kernel = 3, dilation = 2, channels 2d -> d -> d/2 -> d/4, Swish after each,
 * then a per-head linear map to the logit; receptive field 13, the logit of token j is the output at time j + 6
 * (z_j = -inf for j > T-1-6).  Every layer's input is zero at negative times, hidden activations included.
 *   w    = wl0 [H, d, 3, 2d] | wl1 [H, d/2, 3, d] | wl2 [H, d/4, 3, d/2] | wout [H, d/4]    (one fp32 buffer, 16-byte aligned;
 *          wl[o][tau][c] multiplies channel c of the input at time t - (2 - tau) * 2)
 *   bias = bl0 [H, d] | bl1 [H, d/2] | bl2 [H, d/4] | bout [H], or NULL for zero.
 * With bf16 inputs, d = 64 or 32, T > 12 and a workspace of lte_workspace_bytes(LTE_OP_SCORES, s, c) bytes (128-byte
 * aligned; it receives the weights split into bf16 pieces, rebuilt by every call) the stack runs on the tensor cores
 * with exact products and fp32 accumulation; without the workspace, and for every other accepted shape, on the fp32
 * ALUs.  Both agree with an fp64 evaluation to about 1e-5 at |z| of a few units.
 * lte_attn_bwd takes the stack for d = 64 and d = 32: dw and dbias then have the packed layouts of w and bias above.
 * lte_cache_init and lte_attn_decode take the stack for d = 32 or 64 and W >= 20; the step then scores nothing and
 * lte_cache_score has to be called periodically.  lte_attn_bwd_static takes the single layer only.
 */

typedef enum lte_op {
    LTE_OP_SCORES = 0, LTE_OP_SELECT = 1, LTE_OP_PREFILL = 2, LTE_OP_DECODE = 3, LTE_OP_BWD = 4, LTE_OP_CHUNK = 5, LTE_OP_STATS = 6, LTE_OP_CHUNK_STREAM = 7
} lte_op;

/* Bytes of caller-supplied scratch the given entry point needs for this shape (0 if none). */
size_t lte_workspace_bytes(int op, const lte_shape* s, const lte_conv* c);

/*
 * Sticky device-side status of the current device: LTE_OK, or LTE_ERR_DEVICE_STATUS if, since the last call of this
 * function, a kernel gave up on a bounded wait (the outputs of that launch are undefined) or found its input state other
 * than the call said (lte_attn_prefill_chunk, lte_cache_score_unrope describe their cases).  The record is per DEVICE
 * (one word per kernel family), not per cache, workspace or stream: with several caches or streams in flight it tells
 * that something went wrong on the device, not whose launch it was; synchronise and check after the call you care
 * about.  Only the launch that recorded an anomaly is affected: launches made after it, before or after the status is
 * read, wait and run normally.  Synchronous (small copies from the device, ordered after previously launched work by
 * the legacy default stream's rules); reading clears the record.
 */
int lte_device_status(void);

/* Diagnostic (no GPU is touched): initialisations the library's per-device host table has run for ordinal `dev`: 1. */
int lte_selftest_per_device(int dev);

/* Static text for a status code. */
const char* lte_strerror(int status);

/*
 * Retention logits (Section 3.1.1, "LTE module"; the single-layer width-K scorer):
 *   z[b,h,j] = bias[h] + sum_{t<K} sum_{c<2d} w[h,t,c] * x[b,h,j+t-half,c],  x = [k ; v],
 * with x = 0 left of position 0 and no right padding: z = -inf for j > T-1-half (that token's
 * future context does not exist yet).  fp32 accumulation over the exact input values.
 *   k, v      in   [B,H,T,d] of s->dtype
 *   z         out  [B,H,T] fp32
 *   r_or_null out  [B,H,T] fp32 sigmoid(z) (0 where z = -inf), or NULL
 *   ws, ws_bytes   device scratch, used by the three-layer stack only (see lte_conv); may be NULL, 0
 * Errors: INVALID_ARG (NULL or misaligned pointer, K even or > 13, W < K); UNSUPPORTED (n_layers other than 1 or 3,
 * a dilation or kernel other than (1, K) for one layer or (2, 3) for the stack, d not in {32,64,128}, the stack at d = 128).
 */
int lte_scores(const lte_shape* s, const lte_conv* c, const void* k, const void* v,
               float* z, float* r_or_null, void* ws, size_t ws_bytes, void* stream);

/*
 * Capped retention list after a T-token prompt (Eq. 5 restricted to tokens already out of the
 * final window; Section 3.1.3 "Capped capacity": at most R per head, top-R scores on overflow).
 * Candidates: j <= T-1-W with (j < sink or z_j > logit(tau)).  Order: sink positions first, then
 * z descending, ties to the older token.  The first min(R, #candidates) are kept and written in
 * ascending position order.
 *   z             in   [B,H,T] fp32
 *   idx           out  [B,H,R] int32, ascending, unused entries = -1
 *   cnt           out  [B,H]   int32, number kept (<= R)
 *   ncand_or_null out  [B,H]   int32, number of candidates before the cap, or NULL
 * Deterministic and exact on the given z.  Errors: INVALID_ARG; UNSUPPORTED if T-W > 2^24.
 */
int lte_select(const lte_shape* s, const float* z, int32_t* idx, int32_t* cnt,
               int32_t* ncand_or_null, void* ws, size_t ws_bytes, void* stream);

/*
 * The same list interface for the training-free rules the paper's ablation compares with (Section 4, last paragraph:
 * "Unif.+SWA retains out-of-window tokens at a uniform stride"; an eviction heuristic based on accumulated attention):
 *   LTE_RULE_LEARNED     lte_select (score = z).
 *   LTE_RULE_UNIFORM     score is ignored (may be NULL).  Eligible positions are 0 .. E-1, E = max(T - W, 0).  The sink
 *                        positions j < sink come first and count against R; the n = R - #sink remaining slots go to
 *                        sink, sink + stride, sink + 2 stride, ... < E with stride = max(1, ceil((E - sink) / n)), the
 *                        smallest stride that fits.  Every head gets the same list; ncand = E.
 *   LTE_RULE_ACCUM_ATTN  score = a [B,H,T] fp32, the accumulated attention of lte_attn_colsum (or any non-negative
 *                        importance): every position j <= T-1-W is a candidate (no threshold; s->tau is ignored), the R
 *                        largest stay, sink first, ties to the older token.
 * idx, cnt, ncand_or_null as for lte_select.  Errors: INVALID_ARG (unknown rule, NULL score where one is read).
 */
enum { LTE_RULE_LEARNED = 0, LTE_RULE_UNIFORM = 1, LTE_RULE_ACCUM_ATTN = 2 };
int lte_select_rule(const lte_shape* s, int rule, const float* score, int32_t* idx, int32_t* cnt, int32_t* ncand_or_null,
                    void* ws, size_t ws_bytes, void* stream);

/*
 * Accumulated attention of every key under the attention lte_attn_prefill computed (Section 2.2 / Section 4: the quantity
 * eviction heuristics rank by): a[b,h,j] = sum over the queries i with j in A_i, and over the query heads of the group,
 * of exp(scale q_i.k_j - lse_i).  lse is lte_attn_prefill's output for the same q, k, idx, cnt.  The sum of a over j is
 * T * group per head.  A plain fp32 kernel (one warp per key), deterministic; not part of the learned rule's hot path.
 *   q in [B,H*group,T,d], k in [B,H,T,d] of s->dtype;  lse in [B,H*group,T];  a out [B,H,T] fp32
 */
int lte_attn_colsum(const lte_shape* s, const void* q, const void* k, const float* lse, const int32_t* idx, const int32_t* cnt,
                    float* a, void* stream);

/*
 * Prefill attention (Section 3.1.3, "Cached prefilling and decoding"): query i attends over
 * A_i = {max(0,i-W+1) .. i}  U  {j in idx[b,h,:cnt] : j <= i-W}:
 *   o_i = softmax_{j in A_i}(scale * q_i.k_j) v_j,   lse_i = log sum_{j in A_i} exp(scale * q_i.k_j).
 * bf16: tensor-core MMA with fp32 accumulation and fp32 softmax, o rounded to bf16.  fp32: fp32 throughout.
 *   q        in   [B,H*group,T,d] of s->dtype (group = 1 unless s->group says otherwise: query heads
 *                 h*group .. h*group+group-1 attend over key/value head h and its list)
 *   k, v     in   [B,H,T,d] of s->dtype
 *   idx, cnt in   as written by lte_select (idx ascending; entries >= cnt ignored)
 *   o        out  [B,H*group,T,d] of s->dtype
 *   lse      out  [B,H*group,T] fp32 (natural log)
 *   ws       optional device scratch of lte_workspace_bytes(LTE_OP_PREFILL, s, NULL) bytes, 128-byte aligned (bf16, any
 *            supported d): the retained rows idx[:cnt] of k and v are first copied into it as contiguous tensors
 *            [B*H][R][d] (the compaction of Section 3.1.3), and the attention kernel then fetches retained tiles as whole
 *            boxes like the window tiles.  NULL (or too small, or misaligned): the kernel gathers the retained rows itself,
 *            row by row (slower; same results).
 * Errors: INVALID_ARG, UNSUPPORTED (d not in {32,64,128}), CUDA.
 */
int lte_attn_prefill(const lte_shape* s, const void* q, const void* k, const void* v,
                     const int32_t* idx, const int32_t* cnt, void* o, float* lse,
                     void* ws, size_t ws_bytes, void* stream);

/*
 * Decode cache (Fig. 3): per (b,h) a ring of the last W keys/values (slot = position mod W) with
 * their logits, and a pool of at most R retained keys/values with their logits and positions.
 * The cache is one caller-owned device buffer of lte_cache_bytes() bytes; copying it is a
 * checkpoint.  T in the shape is ignored by lte_cache_bytes.
 *
 * Layout: a 256-byte header, then one block per (b,h), padded to a multiple of 256 bytes:
 *   keys    [rows_alloc][d]   rows [0,W) = ring, rows [W,W+R) = pool
 *   values  [rows_alloc][d]
 *   logits  [W+R] fp32, same row order          pool positions [R] int32          {n, cnt, 0, 0} int32
 * rows_alloc = W+R, except for bf16 with d = 64 and W+R <= 256, where rows_alloc = 256 (zero rows at the end) and each
 * key/value row is stored with the 128-byte swizzle (16-byte chunk c of row r sits at chunk position c ^ (r & 7)),
 * which is the layout the tensor-core decode kernel consumes directly from shared memory.
 */
size_t lte_cache_bytes(const lte_shape* s);

/*
 * State after a T-token prompt: ring <- last min(T,W) rows of k, v and their logits from z (the
 * last `half` prompt tokens are still unscored and are scored by the first decode steps), pool <-
 * rows idx[:cnt] of k, v with their logits.  T = 0 gives the empty cache (k, v, z, idx, cnt may
 * then be NULL).  Requires W >= K.
 */
int lte_cache_init(const lte_shape* s, const lte_conv* c, const void* k, const void* v,
                   const float* z, const int32_t* idx, const int32_t* cnt, void* cache, void* stream);

/*
 * One decode step for every (b,h) (Section 3.1.3, decoding paragraph), token n = tokens seen so far:
 *   1. the token leaving the window, p = n-W (if >= 0), is offered to the pool: ignored unless
 *      (p < sink or z_p > logit(tau)); appended if the pool holds fewer than R entries; otherwise it
 *      replaces the lowest-logit entry (the youngest among equals, never a sink entry) iff z_p is
 *      strictly greater;
 *   2. k1, v1 are written to ring slot n mod W;
 *   3. the newest token whose receptive field is now complete, j = n-half, is scored from the ring;
 *   4. o1, lse1 = attention of q1 over the ring (min(n+1, W) entries) and the pool.
 *   cache        in/out
 *   q1           in   [B,H*group,d] of s->dtype;   k1, v1 in [B,H,d]
 *   o1           out  [B,H*group,d] of s->dtype;   lse1 out [B,H*group] fp32
 *   With group > 1 the head's thread block updates the cache (steps 1-3) and then attends for all query heads of the
 *   group over the updated block, which is read once.
 * s->T is ignored.  Errors: INVALID_ARG, UNSUPPORTED (W + R > 4096, d not in {32,64,128}), CUDA.
 */
int lte_attn_decode(const lte_shape* s, const lte_conv* c, void* cache,
                    const void* q1, const void* k1, const void* v1, void* o1, float* lse1,
                    void* stream);

/*
 * Lazy scoring of the ring (Section 3.1.3, "Cached prefilling and decoding": scores are computed in batches, each
 * before its tokens leave the window), for the three-layer stack (lte_conv.n_layers = 3), which lte_attn_decode does
 * not evaluate inside the step: every token in the ring whose receptive field (6 tokens to either side) lies inside
 * the ring, or left of time 0, receives its logit.  A token that is n tokens old can be scored while 7 <= n <= W - 6,
 * and its logit is read when it leaves the window (n = W): call this at least every W - 13 steps; a token that leaves
 * the window unscored is evicted.  Scoring a token again rewrites the same value.
 *   cache      in/out  the state lte_cache_init / lte_attn_decode maintain
 *   ws         device scratch of lte_workspace_bytes(LTE_OP_DECODE, s, c) bytes, 256-byte aligned
 * Errors: UNSUPPORTED for the single layer (it is scored inside the step), INVALID_ARG, WORKSPACE.
 */
int lte_cache_score(const lte_shape* s, const lte_conv* c, void* cache, void* ws, size_t ws_bytes, void* stream);

/*
 * The same for a cache whose keys carry a rotary position embedding (Section 3.1.3, lazy scoring paragraph: the scorer
 * consumes keys as they were before the embedding, the cache stores them after it): the ring's keys are rotated back
 * (the rotation with the sine negated, at each token's own position) on their way into the scorer's input.  Prefill
 * needs nothing of the kind: lte_scores is simply given the un-rotated keys, lte_attn_prefill and lte_cache_init the
 * rotated ones.
 *   rope_cos, rope_sin   in  [rope_len, d/2] fp32 device: cos / sin of the angle of channel pair (c, c + d/2) at position p
 *                        (half-split pairing: (x1, x2) -> (x1 cos - x2 sin, x2 cos + x1 sin) is the embedding);
 *                        both NULL = lte_cache_score
 *   rope_len             positions the tables cover; a ring token at a position >= rope_len keeps its rotated key and
 *                        lte_device_status() reports it
 * Errors: as lte_cache_score; INVALID_ARG for one NULL table or rope_len <= 0.
 */
int lte_cache_score_unrope(const lte_shape* s, const lte_conv* c, void* cache, const float* rope_cos, const float* rope_sin,
                           int32_t rope_len, void* ws, size_t ws_bytes, void* stream);

/*
 * Chunked (continued) prefill on top of a cache (Section 3.1.3, "Cached prefilling and decoding"): T = s->T new tokens
 * arrive at a cache that holds n_past tokens (from lte_cache_init, lte_attn_decode or an earlier chunk).  Chunk-end
 * reading: the pool's entries compete with the tokens that leave the window while the chunk arrives (positions
 * max(n_past - W, 0) .. n_past + T - 1 - W; sink tokens and tokens with z > logit(tau) are candidates); the best R (sink
 * first, then z descending) form the new pool; query i of the chunk sees its window of W keys and the new pool's entries
 * at positions <= i - W.  On top of a one-shot prefill of the first n_past tokens this is exactly the one-shot prefill
 * of the n_past + T tokens, restricted to the chunk's queries; where the cap R never binds it is also what T decode steps
 * compute.  A ring token the cache has not scored yet (the newest K/2 tokens, or whatever lte_cache_score has not
 * reached for the stack) is scored with the chunk as its right context; the chunk's last K/2 tokens stay unscored.
 *   cache    in/out  state for n_past tokens -> state for n_past + T tokens (lte_attn_decode may follow)
 *   n_past   tokens the cache holds, the same for every (b,h); a cache that holds another count is left unchanged and
 *            lte_device_status() reports it
 *   q        in   [B,H*group,T,d];   k, v in [B,H,T,d] of s->dtype
 *   o        out  [B,H*group,T,d];   lse out [B,H*group,T] fp32
 *   ws       device scratch of lte_workspace_bytes(LTE_OP_CHUNK, s, c) bytes, 256-byte aligned: the pool, the ring in
 *            time order and the chunk are laid out as one local sequence of at most R + W + T rows, which the scorer, the
 *            selection and the prefill attention kernels then process (q, o and lse are used in place)
 * Errors: INVALID_ARG, UNSUPPORTED (as lte_cache_init; local sequence too long), WORKSPACE, CUDA.
 */
int lte_attn_prefill_chunk(const lte_shape* s, const lte_conv* c, void* cache, int32_t n_past,
                           const void* q, const void* k, const void* v, void* o, float* lse,
                           void* ws, size_t ws_bytes, void* stream);

/*
 * The same with a choice of reading (flags = 0: lte_attn_prefill_chunk).  LTE_CHUNK_STREAMING: the streaming reading
 * (Section 3.1.3, decoding paragraph, applied token by token inside the chunk): query i of the chunk sees its window and
 * the pool as the replace-the-lowest rule has left it after the token i - W was offered, i.e. exactly what T calls of
 * lte_attn_decode compute, also where the cap R binds: an entry that a later token of the same chunk pushes out is still
 * seen by the queries before that token's.  The cache afterwards is the same under both readings.
 * The pool is walked token by token (one warp per head), which gives every entry that is retained at some query of the
 * chunk and the query from which it is gone.  bf16: the tiled tensor-core kernels attend over that entry list with the
 * leave times as one more mask on their retained tiles (about twice the time of the chunk-end reading); fp32: row by
 * row on the fp32 ALUs (exact as well, but tens of times slower).
 *   ws   device scratch of lte_workspace_bytes(LTE_OP_CHUNK_STREAM, s, c) bytes, 256-byte aligned
 * Errors: as lte_attn_prefill_chunk; INVALID_ARG for unknown flags; UNSUPPORTED for R > 4096 with the flag.
 */
#define LTE_CHUNK_STREAMING 1u
int lte_attn_prefill_chunk_ex(const lte_shape* s, const lte_conv* c, void* cache, int32_t n_past,
                              const void* q, const void* k, const void* v, void* o, float* lse, uint32_t flags,
                              void* ws, size_t ws_bytes, void* stream);

/*
 * Training-side statistics of the scorer (Section 3.1.2, Eq. 7, and the retention count that Algorithm 1 steers):
 *   count[h]  = mean over the batch of #{i : r_i > tau} per sequence          (r = sigmoid(z); the test is z > logit(tau))
 *   penalty   = sum_h lambda[h] sum_{b,i} ReLU(r_i - tau)                     (lambda = 1 when NULL)
 * over the scored positions (z > -inf).  The gradient of the penalty is what lte_attn_bwd adds when given lambda.
 *   z        in   [B,H,T] fp32 device;   lambda_or_null in [H] fp32 device
 *   count    out  [H] fp32 device;       penalty out [1] fp32 device
 *   ws       device scratch of lte_workspace_bytes(LTE_OP_STATS, s, NULL) bytes, 16-byte aligned
 * Fixed summation order (no floating-point atomics).  Errors: INVALID_ARG, UNSUPPORTED (H > 8192), WORKSPACE, CUDA.
 */
int lte_sparsity_stats(const lte_shape* s, const float* z, const float* lambda_or_null, float* count, float* penalty,
                       void* ws, size_t ws_bytes, void* stream);

/*
 * The feedback loop for the penalty weights (Algorithm 1), one call per training step, on HOST arrays of n entries
 * (heads, or layers x heads).  Every call: cbar <- (1 - a) cbar + a count with a = 2 / (1 + period / 2) (the weight of
 * the new sample; the listing prints the two weights the other way round).  When step is a multiple of period:
 * lambda <- lambda alpha if cbar > cap, lambda / alpha if cbar < band cap; lambda <- min(lambda, max); lambda below
 * floor -> 0; cbar > cap with lambda = 0 -> floor.  The listing leaves alpha undefined: 1.2 by default.
 * With several ranks the caller averages `count` (or cbar) over the ranks first, so that every rank takes the same
 * decision ("synchronize" in the listing).  cfg = NULL: period 32, cap 512, alpha 1.2, band 0.95, floor 1e-9, max 1.
 * Pure host arithmetic: no CUDA call, usable without a GPU.  Errors: INVALID_ARG.
 */
typedef struct lte_lambda_cfg {
    int32_t period;                /* u: steps between adjustments                       */
    float cap, alpha, band;        /* retention cap b, adjustment factor, lower band     */
    float floor, max;              /* smallest non-zero weight, upper clamp              */
} lte_lambda_cfg;
int lte_lambda_update(int32_t n, float* lambda, float* cbar, const float* count, int64_t step, const lte_lambda_cfg* cfg);

/*
 * Backward of lte_attn_prefill with the straight-through surrogate (Section 3.1.2):
 *   delta_i = <dO_i, o_i>,  P_ij = exp(scale q_i.k_j - lse_i) on j in A_i,
 *   dV_j = sum_i P_ij dO_i,  dS_ij = P_ij (<dO_i, v_j> - delta_i),
 *   dQ_i = scale sum_j dS_ij k_j,  dK_j = scale sum_i dS_ij q_i;
 *   Eq. 6:  dr_j = <v_j, dV_j>  (+ lambda[h] if z_j > logit(tau), Eq. 7),  dz_j = dr_j r_j (1 - r_j),
 *   for every scored token j <= T-1-half;  dw[h,t,c] = sum_{b,j} dz_j x[b,h,j+t-half,c],
 *   dbias[h] = sum_{b,j} dz_j;  with flags bit 0 the scorer's input gradient
 *   sum_t dz[j-t+half] w[h,t,c] is added into dk (c < d) and dv (c >= d).
 * The retained lists are constants of the backward (the cap is not differentiated).
 *   q,k,v,o,dO in  [B,H,T,d] of s->dtype;  lse, z in [B,H,T] fp32;  idx, cnt as for prefill
 *   lambda_or_null in [H] fp32 device, or NULL
 *   dq,dk,dv   out [B,H,T,d] of s->dtype;  dw out [H,K,2d] fp32;  dbias_or_null out [H] fp32
 * Deterministic (no floating-point atomics).  Errors as for prefill, plus WORKSPACE.
 */
int lte_attn_bwd(const lte_shape* s, const lte_conv* c,
                 const void* q, const void* k, const void* v, const void* o, const float* lse,
                 const void* dO, const float* z, const int32_t* idx, const int32_t* cnt,
                 const float* lambda_or_null,
                 void* dq, void* dk, void* dv, float* dw, float* dbias_or_null, uint32_t flags,
                 void* ws, size_t ws_bytes, void* stream);

#define LTE_BWD_CNN_INPUT_GRAD 1u

/*
 * lte_attn_bwd for callers that cannot hand over scratch memory.  (The paper has no counterpart: this is a
 * deployment convenience of this library.)
 *
 * Who needs it: code that runs where device allocation is off limits or already spent -- a serving process
 * whose memory pool was sized and frozen at start-up, a plugin called from inside another framework's
 * allocator-locked region, or a host that must not call cudaMalloc because that call synchronises the device
 * and would stall every other stream.  Such callers cannot create the workspace lte_attn_bwd asks for.
 *
 * Same arguments and results as lte_attn_bwd, minus `ws` / `ws_bytes` (grouped queries included); the scorer must be
 * the single layer (the three-layer stack answers LTE_ERR_UNSUPPORTED here: its scratch does not fit).  The scratch is a
 * fixed array of LTE_STATIC_SCRATCH_BYTES inside the library; each GPU on which the library's code gets loaded holds
 * it until the process ends.  The call itself performs no cudaMalloc / cudaFree and uses no allocating library routine.
 *   - Shapes whose scratch need (lte_workspace_bytes(LTE_OP_BWD, ...) for flags = LTE_BWD_CNN_INPUT_GRAD; less
 *     without that flag) exceeds LTE_STATIC_SCRATCH_BYTES are rejected with LTE_ERR_WORKSPACE; nothing is launched.
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that device
 *     current).  Under CUDA's lazy loading that look-up is also the moment the driver loads this part of the library
 *     onto the device and sets the array aside, which takes device memory once and may synchronise the device; a
 *     device whose memory is already spent answers LTE_ERR_CUDA.  So make that first call at start-up, before the
 *     memory pool is frozen and outside any stream capture; later calls on that device touch no memory management at all.
 *     cudaDeviceReset() invalidates the looked-up address: do not call this entry point on a device after resetting it.
 *   - All calls on a device share the one array, which still holds whatever the previous call left there.  The
 *     backward kernels write every scratch value before reading it, so no clearing is needed, but two calls that
 *     overlap on the GPU (different streams) would race on it: issue them on one stream, or serialise them.
 */
#define LTE_STATIC_SCRATCH_BYTES (8u << 20)
int lte_attn_bwd_static(const lte_shape* s, const lte_conv* c,
                        const void* q, const void* k, const void* v, const void* o, const float* lse,
                        const void* dO, const float* z, const int32_t* idx, const int32_t* cnt,
                        const float* lambda_or_null,
                        void* dq, void* dk, void* dv, float* dw, float* dbias_or_null, uint32_t flags,
                        void* stream);

#ifdef __cplusplus
}
#endif
#endif /* LTE_H_ */
