/*
 * peagle.h -- C ABI of the B200 (sm_100a) library for P-EAGLE's training-time drafter attention.
 *
 * The operation (paper Section 3, "Scalable Training Framework for Long Contexts"): every
 * length-n sequence is expanded to K parallel-prediction depths, n*K tokens in all.  Token t
 * carries (anchor[t], depth[t]); it sits at sequence position anchor+depth.  A query may attend
 * to a key of the same sequence iff
 *
 *     (depth_k == 0 and anchor_k <= anchor_q)  or  (anchor_k == anchor_q and depth_k <= depth_q)
 *
 * i.e. the real context up to its anchor (Section 2: the depth-0 position is ordinary
 * autoregressive prediction) plus its own chain at the same or earlier depths (Section 3: a
 * depth-d position sees earlier depths only; Section 3.2: position p at depth d depends on
 * position p-1 at depth d-1).  The library evaluates this predicate from the metadata inside
 * its kernels; the (nK)^2 mask the paper pre-computes (Section 3.1) is never stored.
 *
 * Sequence partitioning (Section 3.2, Algorithm 1): attention runs one *query partition* at a
 * time; a partition names its query rows and the keys those rows may see (its own segment plus
 * the depth-0 tokens of earlier segments), and dK/dV are summed in fp32 over the partitions of
 * a sequence (within-sequence gradient accumulation).
 *
 * Conventions for every entry point
 *   - "dev" pointers are CUDA device pointers on the context's device, owned by the caller and
 *     not retained after the call returns.  "host" pointers are ordinary host memory, read
 *     before the call returns.
 *   - Layouts (contiguous, base addresses 16-byte aligned):
 *       Q, O, dO, dQ : bf16 [T][n_q_heads][head_dim]
 *       K, V, dK, dV : bf16 [T][n_kv_heads][head_dim]
 *       LSE          : fp32 [n_q_heads][T], natural-log log-sum-exp of the scaled scores
 *       dK_acc,dV_acc: fp32 [T][n_kv_heads][head_dim]
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Work is enqueued on
 *     it and the call returns without waiting, except where "synchronous" is stated.
 *   - Return value: PEAGLE_OK (0) or a negative peagle_status.  Nothing aborts or throws.
 *     Argument errors are detected on the host before anything is launched.  Errors found on
 *     the device (bad metadata, a wait that ran out) are recorded in a status word that
 *     peagle_poll_status() returns.
 *   - A row whose visible allowed set is empty gets O = 0, LSE = -inf and zero gradients.
 *   - Token order inside a sequence is free; only speed depends on it.
 */
#ifndef PEAGLE_H_
#define PEAGLE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum peagle_status {
    PEAGLE_OK = 0,
    PEAGLE_ERR_NULL = -1,             /* a required pointer is NULL */
    PEAGLE_ERR_BAD_SHAPE = -2,        /* head_dim not 64/128, heads not divisible, K out of [1,255], T mismatch */
    PEAGLE_ERR_BAD_RANGE = -3,        /* range outside its sequence, unsorted or overlapping key ranges */
    PEAGLE_ERR_BAD_META = -4,         /* depth outside [0,K) or anchor outside [0, 2^23) (device-side check) */
    PEAGLE_ERR_UNSUPPORTED_ARCH = -5, /* device is not compute capability 10.x */
    PEAGLE_ERR_WORKSPACE = -6,        /* scratch allocation failed */
    PEAGLE_ERR_TIMEOUT = -7,          /* a bounded device-side wait expired (device-side check) */
    PEAGLE_ERR_TOO_LARGE = -8,        /* request exceeds a documented limit */
    PEAGLE_ERR_CUDA = -9,             /* a CUDA runtime/driver call failed; see peagle_last_cuda_error */
    PEAGLE_ERR_ALIGN = -10            /* a tensor base address is not 16-byte aligned; or (device-side check, head_dim 128
                                         backward) the kernel's shared memory does not start on a 1024-byte boundary */
} peagle_status;

typedef struct peagle_ctx peagle_ctx; /* opaque: device id, scratch memory, device status word */

/* Half-open range of global token indices. */
typedef struct peagle_range {
    int32_t begin, end;
} peagle_range_t;

/* One batch of expanded sequences (Section 3: n x K positions per sequence). */
typedef struct peagle_problem {
    int32_t num_seqs;          /* >= 1 */
    const int32_t *cu_seqlens; /* host [num_seqs+1]: expanded-token offsets, cu[0]=0, non-decreasing */
    int32_t total_tokens;      /* T = cu_seqlens[num_seqs] */
    const int32_t *anchor;     /* dev [T]: index (inside its sequence) of the last real token the chain starts from */
    const int32_t *depth;      /* dev [T]: prediction depth, 0 <= depth < K */
    int32_t K;                 /* number of depths, 1..255 */
    int32_t n_q_heads, n_kv_heads, head_dim; /* n_q_heads % n_kv_heads == 0; head_dim 64 or 128 */
    float softmax_scale;       /* usually 1/sqrt(head_dim) */
} peagle_problem_t;

/* One query partition of one sequence (Algorithm 1: a segment and the keys it may see). */
typedef struct peagle_partition {
    int32_t seq;             /* sequence index */
    peagle_range_t q;        /* query rows, inside sequence `seq`; empty = no-op */
    const peagle_range_t *k; /* host [nk]: visible keys, sorted disjoint non-empty ranges inside `seq` */
    int32_t nk;              /* 0 = the whole sequence is visible; at most 32 ranges, more is
                                PEAGLE_ERR_TOO_LARGE */
} peagle_partition_t;

/* Creates a context on CUDA device `device` (sm_100 only).  Synchronous. */
int peagle_create(peagle_ctx **out, int device);
/* Frees the context and its scratch memory.  Synchronises the device first. */
int peagle_destroy(peagle_ctx *ctx);
const char *peagle_status_string(int status);
/* Text of the last CUDA error the context saw (static storage inside the context). */
const char *peagle_last_cuda_error(const peagle_ctx *ctx);
/* Tile shape the kernels and peagle_classify_tiles use: BM query rows x BN keys. */
int peagle_tile_shape(const peagle_ctx *ctx, int head_dim, int *BM, int *BN);
/* Synchronises `stream`, returns and clears the device status word (PEAGLE_OK,
 * PEAGLE_ERR_BAD_META or PEAGLE_ERR_TIMEOUT).  Synchronous. */
int peagle_poll_status(peagle_ctx *ctx, void *stream);
/* Number of kernels this library has launched through `ctx` since creation. */
int64_t peagle_launch_count(const peagle_ctx *ctx);
/*
 * Measurement hooks (no counterpart in the paper).  With timing on, every later call records a
 * CUDA event pair on its stream around its forward kernel and around its backward kernel.
 * peagle_timing_read synchronises the device, adds up the recorded intervals since the last
 * read, writes ms_out[0] = forward-kernel milliseconds, ms_out[1] = backward-kernel
 * milliseconds, n_out[0], n_out[1] = how many launches of each were timed, and forgets them.
 * At most 4096 launches of each kind are kept between reads; later ones go untimed.
 */
int peagle_timing_enable(peagle_ctx *ctx, int on);
int peagle_timing_read(peagle_ctx *ctx, double *ms_out, int64_t *n_out);

/*
 * Forward of one query partition (Section 3; Algorithm 1 supplies the partition).
 * For every row q in part->q, head h (kv head g = h / (n_q_heads/n_kv_heads)) and visible
 * allowed key set A_q:   s_k = softmax_scale * <Q[q,h], K[k,g]>,
 *   LSE[h][q] = log sum_{k in A_q} exp(s_k),   O[q,h] = sum_k exp(s_k - LSE) V[k,g].
 * Writes O rows and LSE entries of the partition only.  All tensors dev.  The call's tile plan
 * lives in context scratch: concurrent calls on one context from different streams race (use one
 * context per stream).
 */
int peagle_attn_fwd(peagle_ctx *ctx, const peagle_problem_t *prob, const peagle_partition_t *part,
                    const void *Q, const void *K, const void *V, void *O, float *LSE, void *stream);

/*
 * Forward of one query partition for callers that must not allocate device memory.  (The paper
 * has no counterpart: this is a packaging variant of peagle_attn_fwd, same arithmetic, same
 * kernels.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a training step inside a
 * framework whose caching allocator already owns nearly all of the GPU's memory (a raw
 * allocation there fails or makes the framework give its cache back), a latency-critical loop
 * that cannot afford the device-wide synchronisation an allocation implies, or a plug-in host
 * that forbids allocation in its execute callback.  peagle_attn_fwd keeps the tile plan of a
 * call (packed metadata, tile classes, work lists) in context scratch that grows with
 * cudaMalloc; this entry point needs no context and keeps the plan in a fixed array that is
 * part of the library image instead.  It calls no cudaMalloc, cudaFree or any routine that
 * allocates.
 *
 * Cost and limits: the array is PEAGLE_STATIC_SCRATCH_BYTES (4 MiB) of device memory on every
 * GPU that loads the library, held until the process exits.  Accepted sizes:
 * prob->total_tokens <= PEAGLE_STATIC_MAX_TOKENS and (query tiles of the partition) x (key tiles
 * of its visible ranges) <= PEAGLE_STATIC_MAX_TILE_PAIRS, tiles as peagle_tile_shape reports
 * them; anything larger returns PEAGLE_ERR_TOO_LARGE and launches nothing.
 *
 * `device` is the CUDA device ordinal (made current by the call).  The first call on a device
 * looks up the array's device address and the tensor-map encoder, once; make that first call
 * before any stream capture begins.  Work is enqueued on `stream` and the call returns without
 * waiting.  `dev_status` (dev, may be NULL) is one int32 owned by the caller: the call clears it
 * on the stream, and a device-side error (PEAGLE_ERR_BAD_META, PEAGLE_ERR_TIMEOUT) is written
 * there; read it after synchronising the stream.  With dev_status == NULL device-side errors are
 * NOT reported: they go to a word inside the array that no call reads back (bad metadata then
 * shows only as rows that see nothing).
 *
 * All calls on a device share the one array, and it keeps the previous call's contents (the
 * call re-initialises everything it reads).  Two calls whose GPU work overlaps -- different
 * streams, or different host threads -- race on it: keep them on one stream or order them with
 * events.  Q, K, V, O, LSE, prob and part exactly as for peagle_attn_fwd.
 */
#define PEAGLE_STATIC_SCRATCH_BYTES (4u << 20)
#define PEAGLE_STATIC_MAX_TOKENS 32768
#define PEAGLE_STATIC_MAX_TILE_PAIRS 65536
int peagle_attn_fwd_static(int device, const peagle_problem_t *prob,
                           const peagle_partition_t *part, const void *Q, const void *K,
                           const void *V, void *O, float *LSE, int32_t *dev_status, void *stream);

/*
 * Backward of one query partition (Section 3.2: one forward-backward per segment, gradients
 * accumulated across the segments of a sequence).  With P = exp(s - LSE), Delta = <dO, O>,
 * dP_k = <dO[q,h], V[k,g]>, dS_k = P_k (dP_k - Delta):
 *   dQ[q,h]     = softmax_scale * sum_k dS_k K[k,g]              (rows of the partition, written)
 *   dK_acc[k,g] += softmax_scale * sum_{q,h in group g} dS_k Q[q,h]   (ADDED)
 *   dV_acc[k,g] += sum_{q,h in group g} P_k dO[q,h]                   (ADDED)
 * The caller zeroes dK_acc/dV_acc once per sequence.  O and LSE are the forward's outputs for
 * these rows.  Uses context scratch (fp32 dQ staging and Delta); concurrent calls on one
 * context from different streams race.  All tensors dev.
 */
int peagle_attn_bwd(peagle_ctx *ctx, const peagle_problem_t *prob, const peagle_partition_t *part,
                    const void *Q, const void *K, const void *V, const void *O, const void *dO,
                    const float *LSE, void *dQ, float *dK_acc, float *dV_acc, void *stream);

/*
 * The partition driver (Section 3.2 + Algorithm 1): zeroes internal fp32 dK/dV accumulators,
 * then for each partition in the given order runs forward and backward (the partition's LSE is
 * carried from its forward to its backward), and finally rounds the accumulated dK/dV to bf16.
 * Every token of the batch should be a query in exactly one partition.  All tensors dev.
 */
int peagle_attn_partitioned(peagle_ctx *ctx, const peagle_problem_t *prob,
                            const peagle_partition_t *parts, int32_t nparts, const void *Q,
                            const void *K, const void *V, const void *dO, void *O, float *LSE,
                            void *dQ, void *dK, void *dV, void *stream);

/*
 * The driver's two halves for a caller that spreads the query partitions of a batch over several
 * GPUs (Section 3.2: segments are independent given K and V; Section 5.1 trains on 8 GPUs).
 * peagle_attn_partitioned_acc runs forward and backward of the given partitions like the driver
 * but ADDS into the caller's fp32 accumulators dK_acc / dV_acc [T][n_kv_heads][head_dim] (dev,
 * zeroed by the caller) and does not round them.  Each rank calls it with its share of the
 * partitions and the full K / V, the accumulators are summed over the ranks (one collective over
 * the whole arrays; keys that only one rank's queries see add zeros), and peagle_cast_grads rounds
 * the sums to bf16: dK, dV [T][n_kv_heads][head_dim], count = T * n_kv_heads * head_dim (a
 * multiple of 8).  O, LSE and dQ rows belong to the rank that owns their partition.
 */
int peagle_attn_partitioned_acc(peagle_ctx *ctx, const peagle_problem_t *prob,
                                const peagle_partition_t *parts, int32_t nparts, const void *Q,
                                const void *K, const void *V, const void *dO, void *O, float *LSE,
                                void *dQ, float *dK_acc, float *dV_acc, void *stream);
int peagle_cast_grads(peagle_ctx *ctx, const float *dK_acc, const float *dV_acc, int64_t count,
                      void *dK, void *dV, void *stream);

/*
 * The same driver with HOST tensors (pinned memory, or the copies do not overlap anything).
 * K, V and the metadata go to the device first; then every partition's query range is cut into
 * slices of 2,048 rows that are themselves run as query partitions (Section 3.2's scheme: K / V
 * and the fp32 dK / dV sums are shared), so that the copy-in of Q / dO rows, the arithmetic and
 * the copy-out of O / LSE / dQ rows of different slices overlap on three internal streams.  Only
 * rows that belong to a partition are written to O, LSE and dQ.  prob->anchor / prob->depth are
 * HOST pointers for this call only.  Synchronous, also on failure: an error return comes after
 * the internal streams have drained, so nothing writes the caller's buffers afterwards (their
 * contents are then unspecified).  (This is the end-to-end call.)
 */
int peagle_attn_partitioned_host(peagle_ctx *ctx, const peagle_problem_t *prob,
                                 const peagle_partition_t *parts, int32_t nparts, const void *Q,
                                 const void *K, const void *V, const void *dO, void *O, float *LSE,
                                 void *dQ, void *dK, void *dV);

/*
 * Rotary prologue of the drafter layer (Section 2: a LLaMA-3-style layer with rotary position
 * embeddings; Section 3: the token with anchor a and depth d stands at sequence position a + d).
 * qkv is dev [total_tokens][(n_q_heads + 2 n_kv_heads) * head_dim] bf16, one fused projection row
 * per token: query heads, then key heads, then value heads.  Writes the tensors the attention
 * entry points read: Q [T][Hq][D] and K [T][Hkv][D] with every head turned by the rotation of its
 * token's position (element i pairs with element i + D/2; angle = position * rope_base^(-2i/D)),
 * V [T][Hkv][D] copied.  anchor / depth are dev [total_tokens].  All pointers 16-byte aligned;
 * head_dim 64 or 128; rope_base > 1 (LLaMA 3 uses 500000).  Asynchronous on `stream`; nothing is
 * allocated.  Buffers are the caller's; in and out must not overlap.  total_tokens == 0 returns
 * PEAGLE_OK without looking at the pointers; a bad shape or base is PEAGLE_ERR_BAD_SHAPE.
 */
int peagle_rope_qkv_fwd(peagle_ctx *ctx, const void *qkv, const int32_t *anchor, const int32_t *depth,
                        int32_t total_tokens, int32_t n_q_heads, int32_t n_kv_heads,
                        int32_t head_dim, float rope_base, void *Q, void *K, void *V, void *stream);

/*
 * Backward of the prologue: the gradients of Q and K are turned back by the inverse rotation and
 * packed with the gradient of V into d_qkv, the gradient of the fused row (same layout as qkv).
 * Same argument rules as the forward.
 */
int peagle_rope_qkv_bwd(peagle_ctx *ctx, const void *dQ, const void *dK, const void *dV,
                        const int32_t *anchor, const int32_t *depth, int32_t total_tokens,
                        int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, float rope_base,
                        void *d_qkv, void *stream);

/*
 * The projection products of the drafter layer (Section 2: a LLaMA-3-style layer; Section 3.2:
 * every segment runs the layer on its tokens and on the depth-0 tokens before it).  bf16 operands,
 * fp32 accumulation on the tensor cores:
 *     C[m][n] (+)= sum_k A(m, k) * B(n, k),      m < M, n < N, k < K
 * A(m, k) is A[m * lda + k], or A[k * lda + m] when a_transposed; B(n, k) is B[n * ldb + k], or
 * B[k * ldb + n] when b_transposed.  With c_fp32_accumulate == 0, C is bf16 [M][ldc] and is
 * written; otherwise C is fp32 [M][ldc] and the product is ADDED to it (launches on one stream are
 * ordered; two calls that add into the same C from different streams race).  All dev, 16-byte
 * aligned; lda, ldb, ldc (elements) and N multiples of 8; K >= 1.  Elements outside M x N are not
 * touched.  So a linear layer Y = X W^T with W [d_out][d_in] is (A = X, B = W); its input gradient
 * dX = dY W is (A = dY, B = W transposed, K = d_out); its weight gradient dW += dY^T X is
 * (A = dY transposed, B = X transposed, K = rows, fp32 accumulate).  Asynchronous on `stream`.
 */
int peagle_gemm_bf16(peagle_ctx *ctx, const void *A, int64_t lda, int a_transposed, const void *B,
                     int64_t ldb, int b_transposed, void *C, int64_t ldc, int c_fp32_accumulate,
                     int32_t M, int32_t N, int32_t K, void *stream);

/*
 * The attention half of a drafter layer, run segment by segment as Section 3.2 trains long
 * sequences ("Our solution": one forward-backward pass per segment, gradients accumulated across
 * the segments of a sequence; Algorithm 1 phase 3: a segment holds its own tokens and the depth-0
 * tokens before it).  X is dev bf16 [T][d_model], the layer's input rows; W dev bf16
 * [(n_q_heads + 2 n_kv_heads) * head_dim][d_model], the fused query | key | value projection.  For
 * every partition in the given order: the segment's rows are projected (fused rows = X W^T) and
 * rotated (peagle_rope_qkv_fwd); K / V of the visible tokens outside the segment's own block are
 * projected and rotated AGAIN in this segment (they are keys only); the attention forward and
 * backward of the partition run; the segment's dQ, dK, dV go back through the rotation and the
 * projection, and dX, dW are summed in fp32 over the segments and rounded once at the end.
 * Outputs: O [T][n_q_heads][head_dim] bf16 and LSE [n_q_heads][T] fp32 (rows of the partitions
 * only), dX bf16 [T][d_model], dW bf16 like W; dO is the gradient that reaches O.  d_model a
 * multiple of 8; rope_base > 1.  All dev; scratch of about 12 bytes per element of the fused rows
 * is kept in the context.  Asynchronous on `stream`.
 */
int peagle_layer_partitioned(peagle_ctx *ctx, const peagle_problem_t *prob,
                             const peagle_partition_t *parts, int32_t nparts, const void *X,
                             const void *W, int32_t d_model, float rope_base, const void *dO, void *O,
                             float *LSE, void *dX, void *dW, void *stream);

/*
 * Algorithm 1, host only: segment of every token.  `boundaries` is host [S+1], context-token
 * positions with boundaries[0]=0 and boundaries[S]=n (Algorithm 1's B).  Depth 0 and 1 tokens
 * go by their position anchor+depth (a position at or beyond n stays in the last segment);
 * deeper tokens inherit the segment of (anchor, depth-1).  anchor/depth/segment_out are host
 * arrays over the `count` tokens of ONE sequence.  Returns PEAGLE_ERR_BAD_META if a token's
 * dependency (anchor, depth-1) is absent.
 */
int peagle_assign_segments(const int32_t *anchor, const int32_t *depth, int32_t count, int32_t K,
                           const int32_t *boundaries, int32_t S, int32_t *segment_out);

/* ---- test hooks, synchronous ---- */

/*
 * Tile classes of one call (Section 3's mask, looked at BM x BN tiles): query tiles are BM rows
 * from part->q.begin, key tiles BN tokens from the begin of each visible range.
 * host_out[qt * n_ktiles + kt] = 0 SKIP (no allowed pair), 2 FULL (all BN keys present and every
 * in-range row allows all of them), 1 PARTIAL.  host_out may be NULL to query the counts.
 */
int peagle_classify_tiles(peagle_ctx *ctx, const peagle_problem_t *prob,
                          const peagle_partition_t *part, uint8_t *host_out, int32_t *n_qtiles,
                          int32_t *n_ktiles);
/*
 * Self-test of the bounded device-side waits (no counterpart in the paper).  Every wait in the
 * kernels gives up after a time limit, records PEAGLE_ERR_TIMEOUT in the context's status word and
 * lets its CTA return; this call runs that path on purpose: one small CTA waits `limit_ms`
 * milliseconds (1..1000) on a barrier that nothing arrives at.  Returns PEAGLE_OK when the kernel
 * ran to its end; peagle_poll_status() then returns PEAGLE_ERR_TIMEOUT once, and the context stays
 * usable.  Nothing faults or hangs.  Synchronous.
 */
int peagle_selftest_wait_expiry(peagle_ctx *ctx, int32_t limit_ms, void *stream);
/*
 * The mask of one call, materialised by the device predicate: host_out[(q - q.begin) * T + k]
 * for every token k of the batch (1 = allowed and visible).  Only for q_len * T <= 2^26.
 */
int peagle_mask_dense(peagle_ctx *ctx, const peagle_problem_t *prob,
                      const peagle_partition_t *part, uint8_t *host_out);

#ifdef __cplusplus
}
#endif
#endif /* PEAGLE_H_ */
