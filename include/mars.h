/*
 * mars.h -- C ABI of libmars: margin-aware speculative verification (MARS) on one
 * NVIDIA B200 (sm_100a).
 *
 * For every draft position of a batch of speculative-decoding chains or token trees
 * the library streams the target model's logits row over the vocabulary, reduces it
 * to its top-2 (z1, id1, z2, id2), applies the paper's three-way rule, resolves each
 * sequence's longest accepted root-to-node path and emits the accepted length, the
 * accepted tokens and the correction / bonus token.
 *
 * General conventions
 *   - Every pointer is a DEVICE pointer owned by the caller unless a comment says
 *     "host".  The library never allocates, frees or synchronises; it enqueues work on
 *     `cuda_stream` (a cudaStream_t passed as void*, NULL = the default stream) and
 *     returns.  Outputs are valid once the stream has passed that point.
 *   - The return value reports host-detectable errors only; on error nothing is
 *     launched and no output is touched.  Data-dependent problems are reported per
 *     sequence in `seq_status`.
 *   - Layout: B sequences, N rows ("nodes") per sequence, row r = b*N + node; the
 *     logits matrix is [B*N, ld] with row stride `ld` >= V elements; only the first V
 *     elements of a row are read.
 *   - Consecutive calls.  The row-streaming kernels are launched as programmatic dependents of
 *     whatever precedes them on the stream and begin by waiting for it, so by default a call
 *     reads and writes nothing before its predecessor has completed (only its launch latency
 *     overlaps).  With MARS_LOGITS_READY in `flags` the caller vouches that the call's logits do
 *     not come from that predecessor; the call then streams its LOGITS while the predecessor
 *     drains and waits for it only before it reads anything else or writes workspace and
 *     outputs.  This pays where several resident batches are verified back to back (a few
 *     hundred rows: 30 -> 21 us per call); it must not be set when the operation right before the
 *     call on the stream produces, or may still be writing, the call's logits.  Rows may start at any element-aligned address;
 *     16-byte-aligned rows (ld*sizeof(elem) % 16 == 0 and an aligned base) take the
 *     vector path end to end.
 *   - Decisions are taken in fp32: bf16 logits widen exactly, the ratio is one IEEE
 *     round-to-nearest fp32 division, the comparison with theta is strict.
 *   - Total order on a row: larger value first, lower token id first among equal
 *     values (-0 == +0); NaN counts as -inf.  Reported values have -0 replaced by +0.
 */
#ifndef MARS_H_
#define MARS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MARS_OK = 0,
    MARS_ERR_INVALID_ARG = 1, /* NULL required pointer, B<1, N<1, V<2, ld<V, NaN theta, ... */
    MARS_ERR_WORKSPACE = 2,   /* workspace NULL, misaligned (256 B) or too small           */
    MARS_ERR_UNSUPPORTED = 3, /* N or V above the supported caps, unknown dtype / flag      */
    MARS_ERR_CUDA = 4,        /* a CUDA runtime call (memset / launch) reported an error    */
    MARS_ERR_STATIC_CAPACITY = 5 /* mars_verify_tree_static: batch too large for the built-in scratch */
} mars_status_t;

typedef enum { MARS_BF16 = 0, MARS_FP32 = 1 } mars_dtype_t;

/* flags */
#define MARS_SIGN_LITERAL 1u  /* drop the z1 > 0 guard: relax whenever z2/z1 > theta          */
#define MARS_SHARED_PARENT 2u /* `parent` is one [N] array shared by all sequences            */
#define MARS_COUNTERS_ZERO 4u /* mars_verify_chain / _tree: the caller guarantees that the first
                                 4*B bytes of `workspace` are zero, which holds after a
                                 cudaMemset of the workspace and after every completed call of
                                 these functions on it with at least B sequences; the library
                                 then skips its own clearing of those bytes (one stream op less) */

/* Alternative indicators for the relaxation test (the paper's Sec. 3.3 discusses both as the
 * alternatives to its logit ratio; the default, with neither bit set, is the paper's r > theta).
 * With either bit the `theta` argument carries that indicator's threshold, the sign guard and
 * MARS_SIGN_LITERAL do not apply, and everything else (exact match, stop at the first
 * failure, tree resolution) is unchanged.  The two bits are mutually exclusive. */
/* Early start (see "Consecutive calls" above): the caller guarantees that the logits of THIS call
 * were complete before the operation that precedes the call on its stream began -- for instance
 * because that operation is another libmars call on other logits, as when batches that are already
 * resident are verified one after the other.  The call may then stream its logits while its
 * predecessor drains.  Without the bit a call reads nothing before its predecessor on the stream
 * has completed, whatever that predecessor is.  Accepted by mars_verify_chain / _tree / _static,
 * mars_top2_shard and the stochastic calls. */
#define MARS_LOGITS_READY 128u

#define MARS_RULE_MARGIN 8u      /* relax iff Delta = z1 - z2 < theta (fixed logit margin, fp32) */
#define MARS_RULE_PROB_RATIO 16u /* relax iff p2/p1 = exp(z2 - z1) > theta; evaluated as
                                    z1 - z2 < (float)(-ln(theta)), theta <= 0 always relaxes  */

/* Stochastic verification only (mars_verify_tree_stochastic / _chain_stochastic): how the margin
 * rule composes with the acceptance test of Eq. 1.  With neither bit a child that passes the
 * three-way rule is accepted outright and the others take the Eq. 1 test.  Mutually exclusive. */
#define MARS_STOCH_PLAIN 32u      /* Eq. 1 alone: standard speculative sampling, no relaxation  */
#define MARS_STOCH_RELAX_ONLY 64u /* Eq. 1, plus the relaxed runner-up (top-1 is not automatic)  */

#define MARS_MAX_NODES 1024   /* cap on N (rows per sequence)                                 */

/* per-sequence status values written to seq_status */
#define MARS_SEQ_OK 0
#define MARS_SEQ_BAD_TREE 1   /* parent[0] != -1, or for i>0 parent[i] >= i or parent[i] < -1 */
#define MARS_SEQ_DEPTH_CAP 2  /* the accepted path is deeper than Dcap                          */
#define MARS_SEQ_TIMEOUT 3    /* a bounded device-side wait gave up (mars_lmhead_verify only)  */
#define MARS_SEQ_BAD_DISTRIBUTION 4 /* stochastic calls: a row on the walk has no softmax (its
                                       maximum is not finite) or its residual has no mass      */

/* Optional extra outputs; the struct lives in HOST memory, its members are device
 * pointers, any of which may be NULL. */
typedef struct {
    float *top2_val;     /* [B*N, 2]  z1, z2 of every row                                   */
    int32_t *top2_id;    /* [B*N, 2]  id1, id2 of every row                                 */
    uint8_t *node_flags; /* [B, N]    bit0 token == parent's top-1; bit1 token == parent's
                                      top-2 and the parent row relaxes; bit2 accepted (every
                                      ancestor accepted too); bit3 on the emitted path        */
} mars_debug_out_t;

/*
 * Bytes of workspace (device memory, 256-byte aligned) that one call with these sizes
 * needs.  Host function, no CUDA call.  Returns 0 for unsupported sizes.  The workspace
 * holds per-slice top-2 records for rows that are split over several thread blocks and
 * one arrival counter per sequence; its contents need not be initialised or preserved.
 * Two calls that may overlap on the GPU need separate workspaces.
 */
size_t mars_workspace_bytes(int B, int N, int V, mars_dtype_t dt);

/*
 * Chain verification: Algorithm 1 of the paper ("Margin-Aware Speculative Verification
 * Algorithm") with the three-way rule of Sec. 3.4 (exact match / adaptive relaxation
 * r = z(2)/z(1) > theta, Eq. 4 / rejection and correction), plus the bonus token of the
 * Table 1 caption when every draft is accepted.
 *
 *   logits     [B*K, ld] of `dt`; row b*K + i is the target's distribution that judges
 *              draft[b, i]; row K-1 only supplies the bonus token.
 *   draft      int32 [B, K-1]; a negative id or an id >= V never matches.
 *   K          rows per sequence (K-1 drafts), 1 <= K <= MARS_MAX_NODES.
 *   theta      threshold; any non-NaN float; theta >= 1 is strict greedy verification
 *              (Sec. 2.3) unless MARS_SIGN_LITERAL is set.
 *   accept_len int32 [B]    number of accepted drafts a, 0 <= a <= K-1.
 *   out_tokens int32 [B, K] the a accepted drafts followed by the top-1 of row a
 *              (correction if a < K-1, bonus if a == K-1); unused slots are -1.
 *   out_len    int32 [B]    a + 1.
 *   seq_status int32 [B] or NULL; always MARS_SEQ_OK for chains.
 *   dbg        host pointer or NULL.
 */
mars_status_t mars_verify_chain(const void *logits, int64_t ld, mars_dtype_t dt,
                                const int32_t *draft, int B, int K, int V, float theta,
                                uint32_t flags, int32_t *accept_len, int32_t *out_tokens,
                                int32_t *out_len, int32_t *seq_status,
                                const mars_debug_out_t *dbg, void *workspace,
                                size_t workspace_bytes, void *cuda_stream);

/*
 * Tree verification: the same per-token rule (Sec. 3.4) on a token tree (Sec. 2.3,
 * "tree-based methods ... verify many competing prefixes in a single forward pass").
 * Node 0 is the root (the last committed token) and is always accepted.  Node i > 0 is
 * accepted iff its parent is accepted and tok[i] passes the rule against the PARENT's
 * row.  The result is the deepest accepted node, lowest node index among equally deep
 * ones; the emitted next token is the top-1 of that node's row.
 *
 *   logits     [B*N, ld]; row b*N + i is the target's distribution after consuming the
 *              path root -> node i.
 *   tok        int32 [B, N]; tok[., 0] is ignored; negative = padding node.
 *   parent     int32 [B, N] ([N] with MARS_SHARED_PARENT); parent[0] = -1,
 *              parent[i] < i; parent[i] == -1 for i > 0 marks an absent node.
 *   Dcap       capacity of the path outputs; must be >= 0.  If the accepted path is
 *              deeper, the sequence gets MARS_SEQ_DEPTH_CAP and the safe output.
 *   out_tokens int32 [B, Dcap+1]; path_nodes int32 [B, Dcap+1] or NULL (node ids of the
 *              emitted path, root first); unused slots are -1.
 *   seq_status int32 [B] or NULL.  A sequence whose status is not MARS_SEQ_OK gets the
 *              safe output: accept_len 0, out_len 1, out_tokens[0] = top-1 of the root
 *              row, path_nodes[0] = 0, node_flags = {root: accepted|on path, rest 0}.
 */
mars_status_t mars_verify_tree(const void *logits, int64_t ld, mars_dtype_t dt,
                               const int32_t *tok, const int32_t *parent, int B, int N, int V,
                               float theta, uint32_t flags, int32_t *accept_len,
                               int32_t *out_tokens, int32_t *path_nodes, int32_t *out_len,
                               int Dcap, int32_t *seq_status, const mars_debug_out_t *dbg,
                               void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * mars_verify_tree for inputs and outputs that live in HOST memory (the form a caller uses when
 * the logits were not produced on this GPU).  Same rule, outputs and statuses as
 * mars_verify_tree (Sec. 3.4 of the paper; chains are trees with parent[i] = i - 1).  The call
 * enqueues, on `cuda_stream` and in this order: the copies of logits, tokens and parents into the
 * caller's device staging buffer, the verification kernel, and the copies of the results back to
 * the host pointers.  It allocates nothing and does not synchronise: the host buffers must stay
 * valid, and the results are there, once the stream has passed that point.  Pinned host memory
 * makes the copies asynchronous; pageable memory works and is slower.  The step is bound by the
 * host link: B*N*ld*sizeof(elem) bytes cross it per call.
 *
 *   logits_host [B*N, ld]; tok_host [B, N]; parent_host [B, N] ([N] with MARS_SHARED_PARENT)
 *   accept_len_host [B], out_tokens_host [B, Dcap+1], out_len_host [B]        required
 *   path_nodes_host [B, Dcap+1], seq_status_host [B]                          may be NULL
 *   staging      device memory, 256-byte aligned, at least
 *                mars_verify_tree_host_staging_bytes(B, N, V, dt, ld, Dcap) bytes (holds the
 *                device copies of all of the above plus the workspace); contents need not be
 *                initialised; two calls that may overlap need separate staging buffers.
 *   flags        MARS_SIGN_LITERAL, MARS_SHARED_PARENT, MARS_RULE_*.
 * The size query returns 0 for unsupported sizes (host function, no CUDA call).
 */
size_t mars_verify_tree_host_staging_bytes(int B, int N, int V, mars_dtype_t dt, int64_t ld, int Dcap);
mars_status_t mars_verify_tree_host(const void *logits_host, int64_t ld, mars_dtype_t dt,
                                    const int32_t *tok_host, const int32_t *parent_host, int B, int N,
                                    int V, float theta, uint32_t flags, int32_t *accept_len_host,
                                    int32_t *out_tokens_host, int32_t *path_nodes_host,
                                    int32_t *out_len_host, int Dcap, int32_t *seq_status_host,
                                    void *staging, size_t staging_bytes, void *cuda_stream);

/*
 * Bytes of workspace (device memory, 256-byte aligned) for mars_lmhead_verify with these
 * sizes.  Host function, no CUDA call.  Returns 0 for unsupported sizes (d must be a
 * multiple of 64).  Contents need not be initialised or preserved.
 */
size_t mars_lmhead_workspace_bytes(int B, int N, int V, int d);

/*
 * Output projection fused with tree verification: the logits z = W_o h + b_o (Eq. 2 of the
 * paper) are accumulated in fp32 from bf16 operands on the tensor cores and reduced to each
 * row's top-2 inside the GEMM epilogue, so they never reach HBM; the rows' records then go
 * through the same rule and tree resolution as mars_verify_tree.
 *
 *   hidden   bf16 [B*N, d], row-major, 16-byte aligned; row b*N + i is the hidden state
 *            after consuming the path root -> node i.
 *   w_vocab  bf16 [V, d], row-major, 16-byte aligned (W_o).
 *   bias     fp32 [V] or NULL (b_o).
 *   d        hidden size, a multiple of 64.
 *   dbg->top2_val receives the fp32-accumulated logits z1, z2 of every row.
 *   Remaining arguments, outputs and per-sequence statuses are those of mars_verify_tree.
 *   Accumulation order differs from a sequential sum, so near-ties may resolve differently
 *   from an fp64 evaluation; decisions are still taken in fp32 on the accumulated values.
 *   The first call on each device sets function attributes and queries cluster occupancy for
 *   that device (host-side, once per device); make that first call outside any stream capture.
 *   If a bounded device-side wait gives up (which indicates a fault in the pipeline, not a
 *   property of the data), every sequence gets MARS_SEQ_TIMEOUT, accept_len 0, out_len 0 and
 *   out_tokens / path_nodes filled with -1.
 */
mars_status_t mars_lmhead_verify(const void *hidden, const void *w_vocab, const float *bias, int d,
                                 const int32_t *tok, const int32_t *parent, int B, int N, int V,
                                 float theta, uint32_t flags, int32_t *accept_len,
                                 int32_t *out_tokens, int32_t *path_nodes, int32_t *out_len,
                                 int Dcap, int32_t *seq_status, const mars_debug_out_t *dbg,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Exact top-k of logits rows with token ids (1 <= k <= 32, k <= V): the selection a drafter
 * makes when it expands a token tree with the k best continuations of a node (the paper's
 * setup builds its draft trees with top-k = 10, Sec. 4.1).  Same streaming read of each row
 * and the same total order as the verification calls (larger value first, lower id first
 * among equal values, NaN counts as -inf, -0 reported as +0); rows with fewer than k entries
 * above -inf are completed with the lowest unused ids at value -inf.
 *   logits    [rows, ld] of `dt`, first V columns of each row are read.
 *   out_val   float [rows, k], out_id int32 [rows, k]: best first.
 *   workspace mars_topk_workspace_bytes(rows, V, dt, k) bytes, 256-byte aligned; contents need
 *             not be initialised.  One kernel is enqueued when every row is streamed by one
 *             block (from 297 rows on), two when rows are split over several blocks (the
 *             second merges the blocks' lists); nothing is allocated.
 */
size_t mars_topk_workspace_bytes(int64_t rows, int V, mars_dtype_t dt, int k);
mars_status_t mars_topk_rows(const void *logits, int64_t ld, mars_dtype_t dt, int64_t rows, int V,
                             int k, float *out_val, int32_t *out_id, void *workspace,
                             size_t workspace_bytes, void *cuda_stream);

/*
 * Telemetry: histograms of the top-2 statistics that the paper plots for its target models
 * (Fig. 3: top-1 logit values, logit ratios z2/z1, probability ratios p2/p1; Fig. 1 scatters
 * the same quantities), from the [rows, 2] top-2 values a verification call wrote to
 * mars_debug_out_t.top2_val.  No logits are read again.
 *   hist      out, uint32 [3, nbins] (1 <= nbins <= 256), cleared by the call:
 *             [0] z1 over [z1_lo, z1_hi) in nbins equal bins;
 *             [1] r = z2/z1 over [0, 1] for rows with z1 > 0 (r == 1 goes to the last bin);
 *             [2] p2/p1 = exp(z2 - z1) over (0, 1]: bin k holds k/nbins <= p2/p1 < (k+1)/nbins,
 *                 decided as a comparison of z1 - z2 with (float)(-ln(k/nbins)).
 *   outliers  out, uint32 [3]: rows outside the range of the respective histogram (z1 outside
 *             [z1_lo, z1_hi) or not finite; z1 <= 0 or r outside [0, 1] or NaN; z1 - z2 NaN).
 */
mars_status_t mars_top2_histograms(const float *top2_val, int64_t rows, float z1_lo, float z1_hi,
                                   int nbins, uint32_t *hist, uint32_t *outliers, void *cuda_stream);

/*
 * Self-test of the bounded device-side wait used by mars_lmhead_verify's pipeline (the paper
 * has no counterpart).  Launches one block that waits, with the pipeline's own wait routine,
 * on a barrier that nothing ever signals; the wait must give up after `budget_cycles` SM
 * clock cycles (1 .. 2e9) and the kernel must return normally.  Never faults or hangs.
 *   scratch32  32 bytes of device memory, 8-byte aligned; after the stream has passed:
 *              uint32 [0] = MARS_SEQ_TIMEOUT (the status the pipeline would report),
 *              int64 at byte 8 = cycles actually waited, int64 at byte 16 = 0 (wait failed).
 */
mars_status_t mars_selftest_bounded_wait(int64_t budget_cycles, void *scratch32, void *cuda_stream);

/*
 * Read-only streaming probe (the paper has no counterpart; a measurement aid).  Reads `bytes`
 * bytes of device memory once, in chunks of `chunk_bytes` per thread block, with the 16-byte
 * streaming loads and the launch shape of the verification kernel, and keeps only the maximum
 * of the 32-bit words read (atomicMax into *out_max, which the caller zeroes).  Its rate is the
 * ceiling for a kernel that must read every logit; bench.py reports it beside the copy bandwidth.
 *   buffer 16-byte aligned; bytes, chunk_bytes >= 16 (chunk_bytes = one logits row in bench.py).
 */
mars_status_t mars_selftest_stream_read(const void *buffer, size_t bytes, size_t chunk_bytes,
                                        uint32_t *out_max, void *cuda_stream);

/*
 * Vocabulary-parallel verification, step 1 of 2: top-2 of one vocabulary shard.
 * When the logits are sharded over the vocabulary (a tensor-parallel LM head), each rank
 * holds columns [id_offset, id_offset + V_local) of every row.  This call reduces the local
 * shard to one 16-byte record {float z1; int32 id1; float z2; int32 id2} per row, with
 * GLOBAL token ids (local id + id_offset), using the same streaming top-2 (Sec. 3.3 of the
 * paper: top-2 tokens of a logits row) and the same total order as mars_verify_tree.  A
 * record is "unfinished": a shard with fewer than two entries above -inf leaves
 * id = 0x7fffffff in the unused slots; mars_verify_records completes rows after merging.
 *
 *   logits   [B*N, ld] local shard, `dt`; V_local >= 2 columns are read per row.
 *   records  out, [B*N] records, 16-byte aligned device memory.
 *   flags    0 or MARS_COUNTERS_ZERO.
 *   workspace as mars_workspace_bytes(B, N, V_local, dt).
 */
mars_status_t mars_top2_shard(const void *logits, int64_t ld, mars_dtype_t dt, int B, int N,
                              int V_local, int32_t id_offset, void *records, uint32_t flags,
                              void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Vocabulary-parallel verification, step 1 of 2, fused form: the output projection of one
 * vocabulary shard (Eq. 2 of the paper restricted to rows [id_offset, id_offset + V_local) of
 * W_o) reduced to per-row top-2 records inside the GEMM epilogue, as mars_lmhead_verify does,
 * but handed on as records with GLOBAL token ids for mars_verify_records.  Every logit is the
 * same fp32 sum as in the unsharded call, so the merged result is bit-identical to it.
 *   hidden      bf16 [B*N, d] (replicated on every rank); w_shard bf16 [V_local, d];
 *               bias_shard fp32 [V_local] or NULL; d a multiple of 64.
 *   records     out, [B*N] 16-byte records {z1, id1, z2, id2}, 16-byte aligned.
 *   workspace   mars_lmhead_workspace_bytes(B, N, V_local, d) bytes.  After a device-side
 *               timeout (see mars_lmhead_verify) all records are empty (ids 0x7fffffff) and the
 *               first uint32 of the workspace holds MARS_SEQ_TIMEOUT.
 */
mars_status_t mars_lmhead_top2_shard(const void *hidden, const void *w_shard, const float *bias_shard,
                                     int d, int B, int N, int V_local, int32_t id_offset,
                                     void *records, void *workspace, size_t workspace_bytes,
                                     void *cuda_stream);

/*
 * Vocabulary-parallel verification, step 2 of 2: merge the G shard records of every row and
 * verify (three-way rule of Sec. 3.4, tree resolution as mars_verify_tree).  The merge is
 * associative and commutative under the total order, so outputs are bit-identical to
 * mars_verify_tree on the unsharded logits.  Between the two steps the ranks exchange their
 * record arrays (one all-gather of 16 bytes x B*N per rank) into LOCAL memory.
 *
 *   records  [G, B*N] records: shard g's array at records + g*B*N; any shard order.
 *   Other arguments, outputs and statuses as mars_verify_tree (no workspace needed).
 */
mars_status_t mars_verify_records(const void *records, int G, const int32_t *tok,
                                  const int32_t *parent, int B, int N, float theta, uint32_t flags,
                                  int32_t *accept_len, int32_t *out_tokens, int32_t *path_nodes,
                                  int32_t *out_len, int Dcap, int32_t *seq_status,
                                  const mars_debug_out_t *dbg, void *cuda_stream);

/*
 * Stochastic (temperature T > 0) verification of token trees.
 *
 * From the paper: Sec. 2.2 -- a drafted token is accepted with probability
 * min(1, P_target / P_draft) (Eq. 1), a rejection draws the corrected token from the residual
 * distribution, tree-based methods apply the same logic to a token tree, and MARS "modifies only
 * the accept/reject decision" and applies on top of sampling-based verification; Eq. 3 -- P is
 * the softmax of the logits; Sec. 4.1 -- draft trees are top-k expansions.  The paper does not
 * say how the relaxation composes with Eq. 1; the reading implemented here:
 *
 *   - P(v) = softmax(z / T)(v) of a row; NaN logits count as -inf.
 *   - Candidates are deterministic, so the draft distribution at a node is a point mass and
 *     Eq. 1 reads "accept x with probability P(x)".  Starting at the root, the children of the
 *     current node are tried in node order against the current node's row.  A child x is
 *     accepted iff the composition mode accepts it outright (default: x is the row's top-1, or
 *     its runner-up with r > theta -- the three-way rule of Sec. 3.4; see MARS_STOCH_*), or
 *     uniform[b, child] * rem < e_x, where e_x = exp((z_x - max z) / T) and rem is the
 *     unnormalised mass left after removing the siblings rejected so far (the residual of a
 *     point-mass draft is P without that token, renormalised).  The first accepted child
 *     becomes the current node; a repeated sibling token has no mass left.
 *   - When no child is accepted (or the node is a leaf) the next token is drawn from the
 *     residual of the current node's row by inverting its CDF in token-id order with
 *     uniform[b, 0]: the smallest id j with (sum of residual weights of ids <= j) > u * W.
 *   - Arithmetic is fp32 (2^x by the hardware approximation): probabilities carry a relative
 *     error of order 1e-6, so a decision can differ from an exact evaluation only when
 *     |e_x - u * rem| or the distance of u * W to a CDF step is that small relative to the
 *     row's total mass.
 *
 *   logits, tok, parent, B, N, V, theta, Dcap, accept_len, out_tokens, path_nodes, out_len:
 *              as mars_verify_tree; out_tokens[b, a] is the drawn token.
 *   uniform    float [B, N], values in [0, 1): [b, i] judges node i (i > 0), [b, 0] draws the
 *              next token.  Supplied by the caller, so results are reproducible.
 *   temperature T > 0, finite.
 *   flags      MARS_SIGN_LITERAL, MARS_SHARED_PARENT, MARS_RULE_*, MARS_STOCH_*.
 *   seq_status MARS_SEQ_BAD_TREE / MARS_SEQ_DEPTH_CAP: safe output as mars_verify_tree (accept
 *              nothing, emit the root row's top-1).  MARS_SEQ_BAD_DISTRIBUTION: the path so far
 *              is kept and the top-1 of the row where the walk stopped is emitted.
 *   node_prob  float [B, N] or NULL: softmax probability of tok[b, i] under its parent's row
 *              (nothing removed); 0 for the root, absent nodes and ids outside [0, V).
 *   node_how   uint8 [B, N] or NULL: 0 not visited, 1 exact match, 2 relaxed runner-up,
 *              3 accepted by Eq. 1, 4 rejected.
 *   workspace  mars_stochastic_workspace_bytes(B, N, V, dt) bytes, 256-byte aligned; contents
 *              need not be initialised (one 32-byte record per row slice).  Two kernels are
 *              enqueued; nothing is allocated.
 *
 * mars_verify_chain_stochastic is the chain form (K rows, K-1 drafts, uniform [B, K] with
 * [b, i] judging draft i-1 and [b, 0] drawing the correction or bonus token).
 */
size_t mars_stochastic_workspace_bytes(int B, int N, int V, mars_dtype_t dt);
mars_status_t mars_verify_tree_stochastic(const void *logits, int64_t ld, mars_dtype_t dt,
                                          const int32_t *tok, const int32_t *parent,
                                          const float *uniform, int B, int N, int V, float theta,
                                          float temperature, uint32_t flags, int32_t *accept_len,
                                          int32_t *out_tokens, int32_t *path_nodes, int32_t *out_len,
                                          int Dcap, int32_t *seq_status, float *node_prob,
                                          uint8_t *node_how, void *workspace, size_t workspace_bytes,
                                          void *cuda_stream);
mars_status_t mars_verify_chain_stochastic(const void *logits, int64_t ld, mars_dtype_t dt,
                                           const int32_t *draft, const float *uniform, int B, int K,
                                           int V, float theta, float temperature, uint32_t flags,
                                           int32_t *accept_len, int32_t *out_tokens, int32_t *out_len,
                                           int32_t *seq_status, float *node_prob, uint8_t *node_how,
                                           void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Stochastic verification of chains whose drafts were SAMPLED from a drafter's distribution: the
 * acceptance test of Eq. 1 (Sec. 2.2) in its general form.  Draft i was drawn from
 * Q_i = softmax(draft_logits_i / draft_temperature) with probability draft_prob[b, i] = Q_i(draft_i).
 * It is accepted iff the composition mode accepts it outright (as in mars_verify_tree_stochastic)
 * or uniform[b, i+1] * Q_i(x) < P_i(x), which is acceptance with probability min(1, P/Q).  The
 * first rejected position emits a token drawn from the residual distribution
 * norm(max(0, P_i - Q_i)) by CDF inversion in token-id order with uniform[b, 0]; if every draft
 * is accepted, or a negative draft id ends the chain, the token is drawn from P of that row.
 * With MARS_STOCH_PLAIN this is standard speculative sampling.
 *
 *   draft_logits  [B*(K-1), ld_draft], same dtype as `logits`; only the row of the rejected
 *                 position of each sequence is read (twice).
 *   draft_prob    float [B, K-1], the probability with which the drafter drew each draft (the
 *                 drafter knows it; it is not recomputed from draft_logits).
 *   uniform       float [B, K]; other arguments, outputs and statuses as
 *                 mars_verify_chain_stochastic (MARS_SEQ_BAD_DISTRIBUTION also covers a drafter
 *                 row without a softmax and a residual without mass).
 *   workspace     mars_stochastic_workspace_bytes(B, K, V, dt).
 */
mars_status_t mars_verify_chain_sampled(const void *logits, int64_t ld, mars_dtype_t dt,
                                        const void *draft_logits, int64_t ld_draft, const int32_t *draft,
                                        const float *draft_prob, const float *uniform, int B, int K,
                                        int V, float theta, float temperature, float draft_temperature,
                                        uint32_t flags, int32_t *accept_len, int32_t *out_tokens,
                                        int32_t *out_len, int32_t *seq_status, float *node_prob,
                                        uint8_t *node_how, void *workspace, size_t workspace_bytes,
                                        void *cuda_stream);

/*
 * Vocabulary-parallel stochastic verification (a tensor-parallel LM head at T > 0, the setting of
 * the paper's multi-GPU runs: Sec. 4.1, temperature 1, models above 32B on 8 GPUs).  Rank g holds
 * columns [id_offset, id_offset + V_local) of every logits row.  Same reading of Sec. 2.2 / Eq. 1 /
 * Eq. 3 as mars_verify_tree_stochastic; three calls with two exchanges between them:
 *
 *   1. mars_stochastic_shard_records: one streaming pass over the local shard -> per row a
 *      32-byte record {float z1; int32 id1; float z2; int32 id2; float ref; float sum; 8 bytes pad}
 *      (top-2 with GLOBAL token ids, and the shard's softmax mass sum * 2^ref in the scaled
 *      domain z * log2(e) / T), and per node the logit of tok[i] in its parent's row if the shard
 *      holds that column, NaN otherwise.
 *      -- exchange: all-gather records (32 B x B*N per rank) and node logits (4 B x B*N) --
 *   2. mars_stochastic_shard_verify: every rank merges the shards' records, walks the tree
 *      identically (all outputs of mars_verify_tree_stochastic except the drawn token are final
 *      and equal on all ranks), derives from the shards' masses which shard holds the token that
 *      uniform[b, 0] selects from the residual, and only that rank reads its part of the row to
 *      resolve it.  token_part[b] = that token (global id) on the owning rank, -1 on the others;
 *      for sequences without a draw (status not MARS_SEQ_OK) every rank reports the fallback.
 *      out_tokens[b, accept_len[b]] holds the fallback (the row's top-1) until step 3.
 *      -- exchange: all-gather token_part (4 B x B per rank) --
 *   3. mars_stochastic_shard_finish: writes the drawn token into out_tokens[b, accept_len[b]].
 *
 *   records_all [shards, B*N] records, node_logit_all [shards, B*N] floats, token_all [shards, B]:
 *   shard g's array at offset g * (B*N) resp. g * B, in LOCAL memory; my_shard is this rank's
 *   position in them.  shards <= 254.  workspace of step 1:
 *   mars_stochastic_workspace_bytes(B, N, V_local, dt).  Results agree with the unsharded call up
 *   to the rounding of fp32 sums taken in a different order (not bit for bit).
 */
mars_status_t mars_stochastic_shard_records(const void *logits_local, int64_t ld, mars_dtype_t dt,
                                            const int32_t *tok, const int32_t *parent, int B, int N,
                                            int V_local, int32_t id_offset, float temperature,
                                            uint32_t flags, void *records, float *node_logit,
                                            void *workspace, size_t workspace_bytes, void *cuda_stream);
mars_status_t mars_stochastic_shard_verify(const void *logits_local, int64_t ld, mars_dtype_t dt,
                                           const void *records_all, const float *node_logit_all,
                                           int shards, int my_shard, const int32_t *tok,
                                           const int32_t *parent, const float *uniform, int B, int N,
                                           int V_local, int32_t id_offset, float theta, float temperature,
                                           uint32_t flags, int32_t *accept_len, int32_t *out_tokens,
                                           int32_t *path_nodes, int32_t *out_len, int Dcap,
                                           int32_t *seq_status, float *node_prob, uint8_t *node_how,
                                           int32_t *token_part, void *cuda_stream);
mars_status_t mars_stochastic_shard_finish(const int32_t *token_all, int shards, int B, int Dcap,
                                           const int32_t *accept_len, int32_t *out_tokens,
                                           int32_t *seq_status, void *cuda_stream);

/*
 * mars_verify_tree for callers that must not allocate device memory.  (The paper has no
 * counterpart; this is a deployment convenience of the library.)
 *
 * Who needs it: code that runs inside somebody else's memory regime -- an inference server
 * that has handed all free HBM to its KV-cache pool at start-up, a plug-in op inside another
 * runtime, a latency-critical loop where cudaMalloc's implicit device synchronisation is not
 * acceptable.  Such callers cannot create the workspace that mars_verify_tree asks for, so
 * this variant brings its own: a fixed array of mars_static_scratch_bytes() bytes (1 MiB)
 * that is part of the library image.  Every GPU on which the library is loaded holds that
 * array until the process exits, whether or not this function is ever called.
 *
 * The function itself calls no cudaMalloc / cudaFree and no allocating library routine; it
 * issues one cudaMemsetAsync (a few bytes) and one kernel launch on `cuda_stream`, exactly
 * like mars_verify_tree.  Inputs and outputs are still the caller's buffers.
 *
 *   - Capacity: the batch must satisfy mars_workspace_bytes(B, N, V, dt) <=
 *     mars_static_scratch_bytes(); otherwise MARS_ERR_STATIC_CAPACITY is returned and
 *     nothing is launched.  (The serving-scale batch of 256 x 60 rows needs 241 KiB.)
 *   - First call on a device: looks up the array's device address (cudaGetSymbolAddress, with
 *     that device current) and caches it per device.  Make this first call outside any stream
 *     capture.  A failure of the look-up is reported as MARS_ERR_CUDA.
 *   - All calls on one device share the one array.  It keeps whatever the previous call left
 *     in it; the function clears the part that must start at zero (the per-sequence arrival
 *     counters) on the stream before its kernel, on every call: MARS_COUNTERS_ZERO in `flags`
 *     is accepted and ignored here, since no caller can vouch for the contents of an array
 *     that it does not own.  Two calls whose GPU work may overlap --
 *     different streams without an ordering between them, or several host threads -- race on
 *     the array and give undefined results: serialise them, or use mars_verify_tree with
 *     separate workspaces.
 *   - Arguments, outputs and statuses otherwise as mars_verify_tree.
 */
mars_status_t mars_verify_tree_static(const void *logits, int64_t ld, mars_dtype_t dt,
                                      const int32_t *tok, const int32_t *parent, int B, int N,
                                      int V, float theta, uint32_t flags, int32_t *accept_len,
                                      int32_t *out_tokens, int32_t *path_nodes, int32_t *out_len,
                                      int Dcap, int32_t *seq_status, const mars_debug_out_t *dbg,
                                      void *cuda_stream);

/* Size in bytes of the built-in scratch array used by mars_verify_tree_static (host, pure). */
size_t mars_static_scratch_bytes(void);

/*
 * Host: how the current device compares with the one the launch shapes are tuned for.  (The
 * paper has no counterpart.)  Grid sizes, row splits and work-item chunking assume a B200 with
 * 148 SMs; they are pure functions of the call's sizes so that workspace sizes never depend on
 * the device.  On a part with fewer SMs every result stays correct, but waves no longer fill
 * evenly.  *sm_count receives the device's SM count, *sm_tuned 148 (either may be NULL).
 * Returns MARS_OK when they agree and the device is compute capability 10.x,
 * MARS_ERR_UNSUPPORTED when not, MARS_ERR_CUDA if the device cannot be queried.
 */
mars_status_t mars_device_check(int *sm_count, int *sm_tuned);

/*
 * Test hook (the paper has no counterpart; not for deployment): forces a launch shape that the
 * library would not choose by itself, so that tests reach those paths with small inputs.
 * Process-wide, takes effect from the next call, also changes the matching *_workspace_bytes
 * results.  The library never reads the environment: unless this function is called, behaviour
 * depends on the arguments of each call alone.
 *   which 0: slices per logits row (mars_verify_*, mars_top2_shard, mars_topk_rows, stochastic calls)
 *         1: value 1 selects the single-block MMA kernel of mars_lmhead_verify / _top2_shard
 *         2: blocks per cluster of the stochastic tail kernel (1, 2, 4 or 8)
 *         3: value 1 launches every kernel in plain stream order (no programmatic overlap of
 *            consecutive calls; a measurement aid)
 *         4: mars_topk_rows: 1 = 8 vectors per batch and 4 blocks per SM, 2 = 4 vectors per
 *            batch and 6 blocks per SM, whatever the size
 *   value 0 clears the hook.  Returns the previous value, or -1 for an unknown hook / negative value.
 */
int mars_test_hook(int which, int value);

/* Static, human-readable name of a status code (host memory, never NULL). */
const char *mars_status_string(mars_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* MARS_H_ */
