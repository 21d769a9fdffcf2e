/*
 * vocabtrim.h -- C ABI of the B200 (sm_100a) VocabTrim hot path.
 *
 * The library implements the two paths of the method:
 *   offline  : token-frequency counting (Algorithm 1), selection of the K most frequent target
 *              vocabulary ids and reconstruction of the drafter LM head (Eq. 1);
 *   online   : the drafter's trimmed LM head with its token sampling and the index mapper back
 *              to the target vocabulary (Algorithm 2, the drafter-forward and index-mapping steps).
 *
 * Conventions (all entry points unless stated otherwise)
 *   - Every data pointer is a DEVICE pointer owned by the caller.  Entry points whose name ends
 *     in _host take HOST pointers where their comment says so.
 *   - The library allocates no device memory.  The only process-wide state it keeps is host-side
 *     bookkeeping (the launch counter behind vt_launch_count, the calling thread's last CUDA error,
 *     per-device caches of the SM count and of kernel attributes) and the fixed device array of
 *     vt_select_topk_static.  Scratch comes from the caller: `ws` is a device buffer of at least vt_workspace_bytes(op, ...) bytes, 256-byte
 *     aligned, whose first 256 bytes (the control block) must have been cleared ONCE by
 *     vt_workspace_init before its first use.  Every call leaves the control block ready for the
 *     next call.  One workspace serves one stream at a time.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*, NULL = default stream) and
 *     return right after launching.  Argument errors return synchronously without launching.
 *   - Data-dependent problems (token ids outside [0,V), map entries outside [0,V), non-positive
 *     temperatures, NaN rows) never trap and never hang: they set sticky flag bits in the control
 *     block, which vt_read_status reads back.
 *   - bf16 tensors are passed as uint16_t bit patterns, row-major, 16-byte aligned base.
 *   - K is the trimmed vocabulary size (rows of W_trim), V the full target vocabulary, d the
 *     hidden size, B the number of hidden rows per call, topk the candidates per row.
 *   - `map` is in RANK order: map[0] is the most frequent id, ties by count go to the lower id.
 */
#ifndef VOCABTRIM_H
#define VOCABTRIM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    VT_OK = 0,
    VT_ERR_INVALID_ARG = 1, /* null pointer, size out of range, misaligned pointer          */
    VT_ERR_RANGE = 2,       /* data-dependent: ids / map entries out of range (read_status) */
    VT_ERR_WORKSPACE = 3,   /* ws is NULL, misaligned or smaller than vt_workspace_bytes    */
    VT_ERR_CUDA = 4,        /* a CUDA runtime call failed                                   */
    VT_ERR_TIMEOUT = 5,     /* a bounded device-side wait expired (read_status)             */
    VT_ERR_UNSUPPORTED = 6, /* shape outside what the kernels support (see each call)       */
    VT_ERR_NUMERIC = 7      /* data-dependent: non-positive temperature or NaN row          */
} vt_status;

/* Sticky flag bits kept in the workspace control block. */
enum {
    VT_FLAG_BAD_ID = 1u,   /* vt_histogram / vt_build_vocab saw ids outside [0,V); they were skipped */
    VT_FLAG_BAD_MAP = 2u,  /* vt_trim_head saw map entries outside [0,V); those rows were zero-filled */
    VT_FLAG_BAD_TEMP = 4u, /* vt_draft_head saw T <= 0, NaN or Inf; that row reports id -1, logprob NaN */
    VT_FLAG_NAN_ROW = 8u,  /* vt_draft_head produced no finite candidate for a row (NaN inputs)        */
    VT_FLAG_TIMEOUT = 16u  /* a bounded device-side wait expired                                      */
};

/* Operation selectors for vt_workspace_bytes. */
enum {
    VT_OP_HISTOGRAM = 0,
    VT_OP_SELECT_TOPK = 1,
    VT_OP_BUILD_VOCAB = 2,
    VT_OP_TRIM_HEAD = 3,
    VT_OP_DRAFT_HEAD = 4,
    VT_OP_DRAFT_HEAD_HOST = 5,
    VT_OP_BUILD_VOCAB_HOST = 6
};

#define VT_MAX_TOPK 64
#define VT_CTRL_BYTES 256

/* Scratch bytes needed by `op` for the given sizes (arguments an op does not use are ignored).
 * Returns 0 for an unknown op or sizes the op rejects.  Pure host arithmetic. */
size_t vt_workspace_bytes(int op, int64_t n, int32_t V, int32_t K, int32_t d, int32_t B,
                          int32_t topk);

/* Clears the control block (first VT_CTRL_BYTES bytes) of a workspace.  Call once after
 * allocating `ws`, before any other call that takes it. */
vt_status vt_workspace_init(void *ws, size_t ws_bytes, void *stream);

/* Every wait inside the kernels (for a bulk copy to land, for another warp's hand-over) is bounded;
 * when a bound expires the kernel stops waiting, lets its own copies land, raises VT_FLAG_TIMEOUT and,
 * for vt_draft_head, reports every row as id -1 / logprob NaN.  This call sets the bound used by the
 * streaming head kernel of calls that take `ws`: `nanoseconds` of device time per wait, 0 = the
 * built-in default (2 s).  The value stays until changed (vt_workspace_init resets it to 0).
 * Synchronises `stream`.  (No counterpart in the paper: failure handling of this library.) */
vt_status vt_workspace_set_wait_limit(void *ws, uint64_t nanoseconds, void *stream);

/* Synchronises `stream`, copies the sticky flags (VT_FLAG_*) and the count of skipped token
 * ids to the HOST locations `flags` / `n_bad` (either may be NULL), clears them on the device
 * and returns VT_OK, VT_ERR_RANGE (bad ids / map entries), VT_ERR_NUMERIC or VT_ERR_TIMEOUT. */
vt_status vt_read_status(void *ws, void *stream, uint32_t *flags, uint64_t *n_bad);

const char *vt_status_str(vt_status s);

/* Text of the CUDA runtime error behind the calling thread's most recent VT_ERR_CUDA. */
const char *vt_last_cuda_error(void);

/* Number of kernels launched by this library since it was loaded (host counter, for
 * benchmarks that must report their launch count). */
uint64_t vt_launch_count(void);

/*
 * Algorithm 1 (Count Token Frequencies): counts[t] += 1 for every id of the stream.
 *   ids     [n] int32 (any alignment of 4), n >= 0, n < 2^32 per accumulated histogram
 *   counts  [V] uint32; cleared first unless accumulate != 0 (chunked corpora)
 * Ids outside [0,V) are skipped, counted (vt_read_status) and flagged VT_FLAG_BAD_ID.
 * Integer work: the result is exact.
 */
vt_status vt_histogram(const int32_t *ids, int64_t n, int32_t V, uint32_t *counts,
                       int accumulate, void *ws, size_t ws_bytes, void *stream);

/*
 * Measurement aid beside Algorithm 1 (no counterpart in the paper): counts[id mod bins] += 1 for every id
 * inside [0,V), with all `bins` counters (at most VT_FOLDED_MAX_BINS) directly indexed in shared
 * memory as 32-bit words -- a plain walk over the stream (four 128-bit loads in flight per thread) and one
 * shared-memory reduction per token.  An independent, simpler kernel over the same stream: the benchmark
 * reports its rate beside vt_histogram's.  counts [bins] uint32 is cleared first; ids outside [0,V) are
 * skipped silently.  Exact.
 */
#define VT_FOLDED_MAX_BINS 57344
vt_status vt_histogram_folded(const int32_t *ids, int64_t n, int32_t V, int32_t bins, uint32_t *counts,
                              void *stream);

/*
 * Eq. 1, first line: V_trim = V[Top-K(c,k)] from existing counts.
 *   map     [K] int32: map[j] = id of rank j under (count descending, id ascending)
 *   inv_map [V] int32: inv_map[map[j]] = j, -1 for pruned ids
 * 1 <= K <= V.  Integer work: the result is exact and unique.
 */
vt_status vt_select_topk(const uint32_t *counts, int32_t V, int32_t K, int32_t *map,
                         int32_t *inv_map, void *ws, size_t ws_bytes, void *stream);

/*
 * Section 3 (Method) names two selection rules besides Top-K: Top-P and a minimum token frequency.
 * Both cut the same ranking (count descending, id ascending) at a K found from the data:
 *   vt_select_topp    : smallest K whose K most frequent ids hold at least ceil(p * total) of all
 *                       counted tokens, 0 < p <= 1 (evaluated in fp64);
 *   vt_select_minfreq : K = number of ids with count >= min_count.
 * K is clamped to [1, V] and written to the DEVICE int32 *k_out.  map [V]: the first K entries are the
 * trimmed vocabulary in rank order, the entries behind them are not defined (K is not known to the host, so
 * the array must hold V); inv_map [V] is -1 for ranks >= K.
 * Workspace: vt_workspace_bytes(VT_OP_SELECT_TOPK, 0, V, V, ...).  Integer work: exact and unique.
 */
vt_status vt_select_topp(const uint32_t *counts, int32_t V, double p, int32_t *map, int32_t *inv_map,
                         int32_t *k_out, void *ws, size_t ws_bytes, void *stream);
vt_status vt_select_minfreq(const uint32_t *counts, int32_t V, uint32_t min_count, int32_t *map,
                            int32_t *inv_map, int32_t *k_out, void *ws, size_t ws_bytes, void *stream);

/*
 * Draft-tree construction around the head.  Section 4.1 (Settings) adopts the draft-tree construction
 * of EAGLE-2 with depth 3, top-K 8 and at most 32 draft tokens (60 in the depth ablation of the
 * appendix).  The node pool is three caller-owned DEVICE arrays of pool_capacity entries: token id,
 * parent node (-1 = the committed prefix) and cumulative log-probability (fp32).
 *
 * vt_tree_expand: one depth.  Row b of cand_ids / cand_logprobs (DEVICE, row stride ld, candidates in
 * columns col0 .. col0+topk-1: the out_ids / out_logprobs of vt_draft_head fit with ld = 1+topk,
 * col0 = 1) holds the head's top-k for the node frontier_nodes[b] (DEVICE [B], entries < pool_base;
 * NULL, with B = 1, for the first depth whose single row is the committed prefix).  Candidate j of
 * row b becomes node pool_base + b*topk + j with score(parent) + min(logprob, 0) (fp32 addition;
 * score of the prefix is 0).  next_frontier (DEVICE [n_front]) receives the n_front best NEW nodes,
 * best first: higher score, then lower node index; NaN scores rank last.  Hidden row r of the
 * next depth belongs to next_frontier[r].
 *
 * vt_tree_rerank: the final draft.  Of pool nodes [0,n) the `budget` best by the same order are
 * kept and listed in pool order (parents before children): out_nodes (pool index), out_token,
 * out_parent (position in this list, -1 = committed prefix), each DEVICE [budget], padded with -1
 * when n < budget.  Scores never rise along a path, so a kept node's parent is kept (-2 would mark
 * a parent that is not).  The three outputs are the token / parent inputs of vt_verify_greedy.
 *
 * Limits: B*topk and n at most VT_TREE_MAX_NODES (VT_ERR_UNSUPPORTED beyond); n_front <= B*topk and
 * pool_base + B*topk <= pool_capacity (VT_ERR_INVALID_ARG).  Integer results are exact.
 */
#define VT_TREE_MAX_NODES 4096
vt_status vt_tree_expand(const int32_t *cand_ids, const float *cand_logprobs, int32_t B, int32_t topk,
                         int32_t ld, int32_t col0, const int32_t *frontier_nodes, int32_t *pool_token,
                         int32_t *pool_parent, float *pool_score, int32_t pool_base, int32_t pool_capacity,
                         int32_t n_front, int32_t *next_frontier, void *stream);
vt_status vt_tree_rerank(const int32_t *pool_token, const int32_t *pool_parent, const float *pool_score,
                         int32_t n, int32_t budget, int32_t *out_nodes, int32_t *out_token, int32_t *out_parent,
                         void *stream);

/*
 * Greedy verification of S drafted blocks (Section 4, Experiments: the target decodes greedily and a
 * draft token is accepted only if it equals the target's token; the accept loop of Algorithm 2).
 * All pointers are DEVICE pointers, row-major:
 *   token  [S,N]   drafted ids, already full-vocabulary ids (after the index mapper);
 *   parent [S,N]   parent node index, -1 = child of the last committed token; a node whose parent is
 *                  not in [-1, i) is never reached.  NULL = chains (parent[i] = i - 1);
 *   target [S,N+1] target[s,0] = the target's greedy token after the committed prefix,
 *                  target[s,i+1] = its greedy token after the path that ends in node i.
 * From the committed prefix the walk accepts the child of the current node that carries the
 * target's token there (the lowest-indexed one if several do) until no child does.
 *   n_accept [S]      accepted draft tokens per block;
 *   path     [S,N]    accepted node indices, -1 beyond n_accept (may be NULL);
 *   emitted  [S,N+1]  accepted tokens followed by the target's token at the last accepted node,
 *                     -1 beyond (may be NULL); a block yields n_accept + 1 tokens;
 *   tokens_total      DEVICE uint64 the call ADDS sum(n_accept + 1) to (may be NULL); divided by the
 *                     number of blocks it is the block efficiency tau.
 * Integer work: exact.  S = 0 is a no-op.  N < 1 or a NULL required pointer: VT_ERR_INVALID_ARG.
 */
vt_status vt_verify_greedy(const int32_t *token, const int32_t *parent, const int32_t *target, int32_t S,
                           int32_t N, int32_t *n_accept, int32_t *path, int32_t *emitted,
                           uint64_t *tokens_total, void *stream);

/*
 * Memory-bound speed-up of Section 4.1 (Performance Metrics): tau / (c * gamma + 1) with
 * c = draft_params / target_params.  HOST arithmetic in fp64; NaN for arguments outside
 * tau >= 0, draft_params >= 0, target_params > 0, gamma >= 0.
 */
double vt_mbsu(double tau, double draft_params, double target_params, int32_t gamma);

/*
 * vt_select_topk without a workspace.  (The paper has no counterpart: this entry point exists for
 * the sake of callers, not of the method.)  Same result as vt_select_topk, for callers that cannot
 * allocate device memory or pass scratch along: code living inside another runtime's memory pool,
 * processes whose device memory is fully committed at start-up, call sites where the CUDA
 * allocator must not be entered.  The scratch is a fixed array inside the library image:
 * 16 * VT_STATIC_SELECT_MAX_V bytes (2 MiB) held on every GPU that loads the library until the
 * process exits.  No CUDA allocation or free is made by this call, now or later.
 *   - V > VT_STATIC_SELECT_MAX_V returns VT_ERR_UNSUPPORTED; other argument rules as vt_select_topk.
 *   - The first call on each device looks up the array's device address (one synchronous runtime
 *     query, cached afterwards): make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps whatever the last call left in it.
 *     Nothing in it needs clearing between calls (every word is written before it is read), but
 *     two calls whose kernels overlap on the GPU -- different streams, no ordering between them --
 *     race on it and both results are undefined.  Order them on one stream or with events.
 *   - A CUDA failure returns VT_ERR_CUDA (vt_last_cuda_error does not cover this entry point).
 */
#define VT_STATIC_SELECT_MAX_V 131072
vt_status vt_select_topk_static(const uint32_t *counts, int32_t V, int32_t K, int32_t *map,
                                int32_t *inv_map, void *stream);

/* Algorithm 1 followed by Eq. 1, first line: vt_histogram then vt_select_topk (the counts live
 * in the workspace). */
vt_status vt_build_vocab(const int32_t *ids, int64_t n, int32_t V, int32_t K, int32_t *map,
                         int32_t *inv_map, void *ws, size_t ws_bytes, void *stream);

/* Same as vt_build_vocab with `ids` in HOST memory (pinned memory makes the copies
 * asynchronous): the stream is copied to the device in chunks staged in the workspace, each
 * chunk counted as it arrives.  map / inv_map stay device pointers. */
vt_status vt_build_vocab_host(const int32_t *ids_host, int64_t n, int32_t V, int32_t K,
                              int32_t *map, int32_t *inv_map, void *ws, size_t ws_bytes,
                              void *stream);

/*
 * Eq. 1, second line: W_trim = W[Top-K(c,k), :], a bit copy of K rows.
 *   W_full [V,d] bf16, W_trim [K,d] bf16, d % 8 == 0, map [K] int32.
 * `ws` may be NULL; when given, map entries outside [0,V) are flagged VT_FLAG_BAD_MAP.  Such rows
 * are zero-filled either way.
 */
vt_status vt_trim_head(const uint16_t *W_full, const int32_t *map, uint16_t *W_trim, int32_t V,
                       int32_t K, int32_t d, void *ws, void *stream);

/*
 * Algorithm 2 (drafter forward over the trimmed head, then the index mapping), head part: logits = h W_trim^T (bf16 inputs, fp32 accumulation),
 * z = logits / T_b, log-softmax statistics, the `topk` best candidates per row, a Gumbel-max
 * draw argmax_j (z_j - log(-log u_bj)) and the index mapper T_{d->t} (trimmed index -> target id).
 * Logits never leave the chip.
 *   h        [B,d]  bf16            W_trim  [K,d] bf16
 *   map      [K] int32 or NULL (identity: the untrimmed head)
 *   temp     [B] fp32, T_b > 0      uniforms [B,K] fp32 or NULL (no sampling)
 *   out_ids      [B, 1+topk] int32: column 0 = sampled id (greedy id if uniforms == NULL),
 *                                   columns 1.. = candidates in descending z, ties to lower index
 *   out_logprobs [B, 1+topk] fp32 : log softmax(logits/T_b) of the id in the same column
 * Uniforms are clamped to [2^-24, 1-2^-24].  Limits: d % 8 == 0, 1 <= topk <= min(K, 64),
 * 1 <= B <= 256.  B <= 16 with d <= 8192 (B <= 8) or d <= 4096 runs the streaming kernel; every
 * other shape runs the dense tensor-core kernel, which keeps its top-k lists in registers and
 * takes topk <= 16 (VT_ERR_UNSUPPORTED beyond).
 */
vt_status vt_draft_head(const uint16_t *h, const uint16_t *W_trim, const int32_t *map, int32_t B,
                        int32_t K, int32_t d, const float *temp, int32_t topk,
                        const float *uniforms, int32_t *out_ids, float *out_logprobs, void *ws,
                        size_t ws_bytes, void *stream);

/*
 * vt_draft_head for drafting loops (Algorithm 2's inner loop runs the head once per draft token):
 * same arguments and results, but the kernel is launched so that it may become resident and start
 * fetching W_trim while work enqueued earlier on the stream is still finishing (programmatic
 * dependent launch); it reads h, temp, uniforms, map and the workspace only after that earlier work
 * has completed.  The caller promises that W_trim was not written by work still pending on the
 * stream -- weights are static while drafting; after vt_trim_head, synchronise or make one plain
 * vt_draft_head call first.  Both kernels take part: the dense kernel's first ring of W_trim tiles is
 * requested early as well, and its merge kernel is chained the same way.
 */
vt_status vt_draft_head_overlapped(const uint16_t *h, const uint16_t *W_trim, const int32_t *map,
                                   int32_t B, int32_t K, int32_t d, const float *temp, int32_t topk,
                                   const float *uniforms, int32_t *out_ids, float *out_logprobs,
                                   void *ws, size_t ws_bytes, void *stream);

/*
 * One tree depth in one call: vt_draft_head_overlapped followed by vt_tree_expand on its candidates
 * (out_ids / out_logprobs columns 1..topk), with the same arguments, results and limits as those two
 * (Algorithm 2, the drafter-forward and index-mapping steps with the draft tree of Section 4.1).  For the streaming kernel's shapes
 * (B <= 16) the expansion runs inside the head kernel, in the CTA that merges the rows, so a tree
 * depth costs one launch; other shapes chain the expansion kernel behind the merge.  The caller's
 * promise about W_trim is that of vt_draft_head_overlapped.
 */
vt_status vt_draft_head_expand(const uint16_t *h, const uint16_t *W_trim, const int32_t *map, int32_t B,
                               int32_t K, int32_t d, const float *temp, int32_t topk,
                               const float *uniforms, int32_t *out_ids, float *out_logprobs,
                               const int32_t *frontier_nodes, int32_t *pool_token, int32_t *pool_parent,
                               float *pool_score, int32_t pool_base, int32_t pool_capacity, int32_t n_front,
                               int32_t *next_frontier, void *ws, size_t ws_bytes, void *stream);

/* Parity-only variant of vt_draft_head: also writes the fp32 logits [B,K] and lse [B]
 * (log sum exp of z) when those pointers are non-NULL.  Never used for timing. */
vt_status vt_draft_head_debug(const uint16_t *h, const uint16_t *W_trim, const int32_t *map,
                              int32_t B, int32_t K, int32_t d, const float *temp, int32_t topk,
                              const float *uniforms, int32_t *out_ids, float *out_logprobs,
                              void *ws, size_t ws_bytes, void *stream, float *out_logits,
                              float *out_lse);

/* Same as vt_draft_head with the per-step tensors in HOST memory: h, temp, uniforms are copied
 * in and out_ids, out_logprobs copied back through staging areas in the workspace, all on
 * `stream`; the call returns after enqueueing (synchronise the stream before reading the
 * outputs).  W_trim and map are the resident model state and stay DEVICE pointers.  temp,
 * out_ids and out_logprobs in page-locked (pinned) host memory are read and written in place by
 * the kernels instead of being copied; pageable buffers work too and take the staging route. */
vt_status vt_draft_head_host(const uint16_t *h_host, const uint16_t *W_trim, const int32_t *map,
                             int32_t B, int32_t K, int32_t d, const float *temp_host,
                             int32_t topk, const float *uniforms_host, int32_t *out_ids_host,
                             float *out_logprobs_host, void *ws, size_t ws_bytes, void *stream);

#ifdef VT_STAMPS
/*
 * Instrumented builds only (compiled with -DVT_STAMPS; the regular library does not export it).  The
 * streaming head kernel then writes a nanosecond clock stamp per CTA at fixed phases of Algorithm 2's
 * head step (entry, ring requested, released by the launch dependency, first stage landed, last stage
 * consumed, record written, fence, ticket, merge loads / selection / outputs) into the workspace:
 * 8-byte words [max_ctas][slots] at byte `offset` of `ws`.  Returns 0 for shapes the streaming kernel
 * does not take.  Pure host arithmetic.
 */
int32_t vt_stamps_region(int32_t B, int32_t d, int32_t topk, size_t *offset, int32_t *slots, int32_t *max_ctas);
#endif

#ifdef __cplusplus
}
#endif
#endif /* VOCABTRIM_H */
