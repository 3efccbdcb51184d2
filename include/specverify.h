/*
 * specverify.h -- C ABI of libspecverify: batched verification of a draft token tree on one GPU.
 *
 * The library implements the verification step of multi-path speculative decoding (paper
 * Section 2, step 3): given target and draft logits on the nodes of a draft tree, the tree, the
 * sampling parameters and caller-supplied uniforms, it selects one accepted node and one
 * correction ("bonus") token so that the emitted tokens follow the target distribution.
 *
 * General rules for every entry point
 *   - `extern "C"`, plain pointers and sizes.  Unless a parameter says "host", a data pointer is
 *     a DEVICE pointer owned by the caller; the library only borrows it until the work it
 *     enqueued on `stream` has finished.  `SpecIn` / `SpecOut` themselves are host structs, read
 *     during the call only.
 *   - `stream` is a `cudaStream_t` passed as `void*` (NULL = the legacy default stream).  Calls
 *     enqueue kernels and return; they never synchronise, allocate or free.
 *   - Scratch memory comes from the caller: `ws` (device, 256-byte aligned) of at least
 *     `spec_workspace_bytes()` bytes.  Two calls that may overlap on the GPU need two workspaces.
 *   - Return value: SPEC_OK or a negative SPEC_ERR_* found on the host before anything was
 *     enqueued.  Problems only visible on the device (bad topology or token, a non-finite row, a
 *     bounded wait that ran out) are reported per sequence in `SpecOut.status` (a SPEC_DEV_*
 *     code); that sequence gets accept_len = -1 and accepted_node = -1.  Nothing traps.
 *   - There is no CPU fallback.
 *
 * Tree layout (Definition 3.1, Definition 5.2): node 0 is the root (the current context);
 * parent[0] = -1 and parent[i] < i.  The child list of a node is the set of nodes naming it as
 * parent, in increasing index order; that is the order in which children are tried.  Equal tokens
 * under one parent stay separate nodes (multiplicity, Section 3.2).  At most SPEC_MAX_CHILDREN
 * children per node and SPEC_MAX_NODES nodes per sequence.
 *
 * Sampling distribution of a row (Section 4 names temperature and nucleus sampling; top-k is an
 * addition): y = z / T, softmax; top-k keeps every token whose logit is >= the k-th largest logit
 * value; top-p then keeps the fewest leading groups of equal-logit tokens whose mass (within the
 * top-k set) reaches top_p; renormalise.  The same transform is applied to target and draft rows.
 */
#ifndef SPECVERIFY_H
#define SPECVERIFY_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPEC_MAX_CHILDREN 16
#define SPEC_MAX_NODES 1024

/* host-side return codes */
#define SPEC_OK 0
#define SPEC_ERR_NULL (-1)        /* a required pointer is NULL                                  */
#define SPEC_ERR_SHAPE (-2)       /* B, N, V or a stride is out of range                         */
#define SPEC_ERR_DTYPE (-3)       /* logits_dtype is neither SPEC_F32 nor SPEC_BF16              */
#define SPEC_ERR_PARAM (-4)       /* temperature <= 0 or not finite, top_p outside (0,1], top_k < 0 */
#define SPEC_ERR_WORKSPACE (-5)   /* ws NULL, misaligned or too small                            */
#define SPEC_ERR_UNSUPPORTED (-6) /* vocabulary too large for the on-chip plan of this device    */
#define SPEC_ERR_CUDA (-7)        /* a CUDA runtime call failed (launch configuration, no device) */

/* per-sequence device status codes (SpecOut.status) */
#define SPEC_DEV_OK 0
#define SPEC_DEV_TOPOLOGY 1       /* parent[0] != -1, parent[i] outside [0,i), too many children */
#define SPEC_DEV_TOKEN 2          /* token outside [0,V)                                         */
#define SPEC_DEV_NONFINITE 3      /* a logit row holds NaN / +inf, or only -inf                  */
#define SPEC_DEV_TIMEOUT 4        /* a bounded on-device wait ran out                            */

#define SPEC_F32 0
#define SPEC_BF16 1

typedef struct {
    int32_t B, N, V;              /* sequences, nodes per sequence (root included), vocabulary   */
    int32_t logits_dtype;         /* SPEC_F32 or SPEC_BF16                                        */
    const void *target_logits;    /* [B,N,V] row of node a of sequence b at b*seq_stride + a*node_stride */
    const void *draft_logits;     /* same layout; rows of nodes without children are never read  */
    int64_t seq_stride;           /* in elements                                                  */
    int64_t node_stride;          /* in elements, >= V; the V entries of a row are contiguous     */
    const int32_t *parent;        /* [N], or [B,N] with topo_seq_stride = N                       */
    int64_t topo_seq_stride;      /* 0: one topology shared by the batch                          */
    const int32_t *token;         /* [B,N] draft token of each node; token[b,0] is ignored        */
    float temperature;            /* > 0                                                          */
    int32_t top_k;                /* 0 = off                                                      */
    float top_p;                  /* in (0,1]; 1 = off                                            */
    const float *temperature_per_seq; /* optional [B]; overrides `temperature` when not NULL      */
    const float *u_accept;        /* [B,N] uniforms in [0,1): entry of node a decides a's test    */
    const float *u_bonus;         /* [B,N] uniforms in [0,1): the stop node's entry draws the bonus */
} SpecIn;

typedef struct {
    int32_t *accepted_node;       /* [B] index of the accepted node (0 = nothing accepted)        */
    int32_t *accept_len;          /* [B] tau = depth of the accepted node                          */
    int32_t *out_tokens;          /* [B,N] tokens on the accepted path, then the bonus, then -1   */
    int32_t *bonus_token;         /* [B]                                                           */
    int32_t *status;              /* [B] SPEC_DEV_*                                                */
    /* optional outputs: skipped when NULL */
    float *residual;              /* [B,V] the distribution the bonus token was drawn from         */
    float *node_thr;              /* [B,N] threshold node a is tested with as if it were reached:
                                     SpecInfer: min(1, P/q) after its earlier siblings were rejected
                                     (asking for it disables the early exit after an accepted
                                     sibling); Traversal: the final weight of a.  Root: 1          */
    float *node_w_in;             /* [B,N] Traversal only: weight handed to a by its parent        */
    float *node_features;         /* [B,N,4] entropy (nats) of the target and draft sampling
                                     distributions and their largest probability:
                                     H_p, H_q, top1_p, top1_q (q entries 0 for childless nodes)   */
    float *margin;                /* [B,N+1] |u_accept - threshold| per node (NaN where the node
                                     was not evaluated), last entry: distance of the bonus draw to
                                     the nearer CDF boundary, as a fraction of the total mass      */
} SpecOut;

/* Bytes of scratch the calls below need for these shapes (depends on B, N only).
 * host pointers.  Returns SPEC_OK or SPEC_ERR_NULL / SPEC_ERR_SHAPE. */
int32_t spec_workspace_bytes(const SpecIn *in, int64_t *bytes);

/*
 * Sampling distribution of every node's target (which = 0) or draft (which = 1) row, written to
 * HBM (Section 4: temperature / nucleus; tie rules above).
 *   probs      [B,N,V] float, contiguous.  May be NULL when only the statistics are wanted.
 *   row_stats  optional [B,N,6] float: max of z/T, sum of kept exp(z/T - max), kept count,
 *              entropy (nats), largest probability, smallest kept logit value.
 * Only B, N, V, dtype, the logits of the chosen side, strides and the sampling parameters of `in`
 * are read (every row of the chosen side is read, whatever the tree).  With truncating parameters
 * (top_k or top_p active) `ws` must be a workspace of spec_workspace_bytes(); otherwise it may be
 * NULL.  Rows that are not finite produce NaN statistics and zero probabilities.
 */
int32_t spec_tree_probs(const SpecIn *in, int32_t which, float *probs, float *row_stats,
                        void *ws, int64_t ws_bytes, void *stream);

/*
 * The first half of a verification call on its own: the statistics (reference, normaliser, top-k /
 * top-p cut) of every row the verifiers read -- the one pass over the logits in HBM (Section 4's
 * sampling transform, without materialising the distributions).  Results stay in `ws`; the entry point
 * exists so that this pass can be timed and profiled by itself.  Same arguments and checks as the
 * verifiers.
 */
int32_t spec_row_statistics(const SpecIn *in, void *ws, int64_t ws_bytes, void *stream);

/*
 * SpecInfer verification (Algorithm 4 used top-down, Section 3.2 "OT-based algorithms"):
 * starting at the root, try the children of the current node in list order; child x is accepted
 * when u_accept < min(1, P(x)/q(x)), where P is the node's target distribution after the residual
 * updates P <- norm((P - q)+) of the siblings rejected before it; on acceptance move to that
 * child, otherwise stop and draw the bonus token from P by inverse CDF with the node's u_bonus
 * (from the unmodified target distribution at a childless node).
 * Fused: logits in, decisions out; no [B,N,V] tensor is written.
 */
int32_t spec_verify_specinfer(const SpecIn *in, const SpecOut *out, void *ws, int64_t ws_bytes,
                              void *stream);

/*
 * Top-down verification with one of the other OTLP solvers the paper defines (Appendix B; composed as
 * Section 3.2 "OT-based algorithms" says: at a node the solver puts out one token; the walk moves to the
 * first child, in list order, that carries it, and stops when no child does -- that token is the
 * correction token).  solver: 0 = NSS (Algorithm 1: the token is drawn from p, the drafts are ignored),
 * 1 = NaiveTree (Algorithm 2: the first child is tested with min(1, p/q), otherwise a draw from
 * norm((p - q)+)), 2 = SpecTr K-SEQ (Algorithm 3: division factor rho* by bisection, every child
 * tested with min(1, p / (rho q)), otherwise a draw from its residual).  A child's test uses its entry
 * of u_accept, a draw at node a the entry u_bonus[a].  Same inputs, workspace, stream and status rules
 * as spec_verify_specinfer; of SpecOut only accepted_node, accept_len, out_tokens, bonus_token and
 * status are written, and the optional outputs must be NULL (SPEC_ERR_UNSUPPORTED otherwise, and for
 * N > 128).  solver outside 0..2: SPEC_ERR_PARAM.
 */
int32_t spec_verify_otlp(const SpecIn *in, const SpecOut *out, int32_t solver, void *ws, int64_t ws_bytes,
                         void *stream);

/*
 * SpecInfer verification for callers that cannot allocate device memory.  The paper has no
 * counterpart to this entry point: it exists for hosts of this library that are handed their
 * device buffers by someone else and may not call cudaMalloc themselves -- a plugin running inside
 * an inference server whose memory pool is closed to it, a process under a fixed memory budget, or
 * code that runs where an allocation would stall or fail (a latency-critical decoding loop, a
 * region in which the allocator is locked).  Same inputs, outputs and results as
 * spec_verify_specinfer, but no `ws` argument: the scratch memory is an array of
 * SPEC_STATIC_WS_BYTES bytes inside the library image, present on every GPU that has loaded the
 * library until the process exits.
 *   - Limit: B * N <= SPEC_STATIC_MAX_NODES (tree nodes summed over the batch); larger shapes
 *     return SPEC_ERR_WORKSPACE and nothing is enqueued.  V is not limited by the scratch.
 *   - The first call on a device looks up the array's device address (once per device, with that
 *     device current) before it enqueues anything; make that first call outside any stream
 *     capture.  No call allocates or frees memory.
 *   - Every call uses the same array, which still holds the previous call's records when the next
 *     one starts; the call clears the parts that must start empty (the published weights and the
 *     arrival counters) on `stream` itself.  Two calls that can overlap on the GPU (different
 *     streams without an ordering between them) race on the array: serialise them, or give the
 *     others a workspace through spec_verify_specinfer.
 */
#define SPEC_STATIC_MAX_NODES 4096
#define SPEC_STATIC_WS_BYTES (1536 * 1024)
int32_t spec_verify_specinfer_static(const SpecIn *in, const SpecOut *out, void *stream);

/*
 * Traversal Verification (Section 3.2, bottom-up; block verification of Section 3.1 on one
 * path).  Weights flow down: a child with token x gets min(1, w P(x)/q(x)) from its parent's
 * current (w, P); a node is tested (u_accept < w) only after all its child subtrees were
 * rejected, each rejection updating the parent to S = sum (wP - q)+, w <- S / (S + 1 - w),
 * P <- (wP - q)+ / S.  The first node accepted in depth-first post-order wins; the root always
 * accepts.  The bonus token is drawn from the accepted node's final P with its u_bonus.
 */
int32_t spec_verify_traversal(const SpecIn *in, const SpecOut *out, void *ws, int64_t ws_bytes,
                              void *stream);

/*
 * Offline analysis of a batch of draft trees (Section 5 and Appendices C, D): for every node with
 * children, from its sampling distributions p, q (same transform as the verifiers) and its child list,
 *   acceptance  [B,N,4] acceptance rates alpha(f) of Definition 5.1 with k = the node's number of
 *               children: NSS (Algorithm 6), Naive (Algorithm 7), SpecTr (Algorithm 8), SpecInfer
 *               (Algorithm 9);
 *   divergence  [B,N,3] L1 distance sum |p - q| (Section 5), KL(p||q), KL(q||p) in nats (the selector's
 *               scalar features, Section 6; +inf where the second law has no mass under the first);
 *   branch      [5][B,N] branching probability B(f, ch(parent), token) of Definition 5.3 of moving from
 *               the parent into the node, for f = NSS (Algorithm 11), Naive (12), SpecTr (13), SpecInfer
 *               with children tried in list order (what spec_verify_specinfer runs), SpecInfer with the
 *               next child picked uniformly (Algorithm 14; NaN for more than 10 children); root: 1; a
 *               child whose token an earlier sibling carries is never moved to: 0;
 *   reach       [5][B,N] product of the branching probabilities along the node's path;
 *   block_eff   [5][B]  sum of reach over the tree's nodes = E[tau + 1 | tree], the inner sum of
 *               equation (3) (average it over sampled trees for the paper's estimator).
 * Rows of childless nodes are NaN in acceptance / divergence.  All outputs are device pointers, all
 * required.  `ws`: spec_analysis_workspace_bytes() bytes.  u_accept / u_bonus of `in` must be valid
 * but do not influence the outputs.  SpecTr's rho* is found by 40 bisection steps on [1, k].
 */
typedef struct {
    float *acceptance;
    float *divergence;
    float *branch;
    float *reach;
    float *block_eff;
} SpecAnalysisOut;
int32_t spec_analysis_workspace_bytes(const SpecIn *in, int64_t *bytes);
int32_t spec_tree_analysis(const SpecIn *in, const SpecAnalysisOut *out, void *ws, int64_t ws_bytes, void *stream);

/*
 * Forward-pass time of delayed-expansion actions (Appendix E, equation (8)): for action a = (K, L1, L2)
 * at context length ctx,
 *   T_hat[a] = sum_{j<L1} t_q(ctx + j) + sum_{j<L2} t_q(ctx + L1 + j K) + t_p(ctx + L1 + K L2),
 * t_q / t_p: measured draft / target forward times per context length (tables of n_len doubles; a length
 * beyond the table uses its last entry).  actions [n_actions,3] int32, T_hat [n_actions] double; all
 * device pointers.
 */
int32_t spec_latency_model(const double *t_q, const double *t_p, int32_t n_len, int32_t ctx, const int32_t *actions,
                           int32_t n_actions, double *T_hat, void *stream);

/*
 * Inverse-CDF draw (the "Sample Y ~ p" steps of Algorithms 1-4) from R rows of non-negative
 * weights that need not be normalised: token[r] = smallest t with w_0 + ... + w_t > u[r] * sum(w).
 *   weights [R,V] float contiguous, u [R] in [0,1), token [R] (-1 for an all-zero row),
 *   margin optional [R]: distance to the nearer CDF boundary as a fraction of the total.
 */
int32_t spec_sample_bonus(const float *weights, int32_t R, int32_t V, const float *u,
                          int32_t *token, float *margin, void *ws, int64_t ws_bytes, void *stream);

/*
 * Host-buffer form of the two verifiers (the verification step of Section 2 for a caller whose
 * logits sit in host memory).  Every data pointer of `in` and `out` is a HOST pointer (pinned
 * memory gives asynchronous copies); logits must be dense ([B,N,V] contiguous).  `dev_buf` is a
 * DEVICE buffer of at least spec_host_staging_bytes() bytes, 256-byte aligned, owned by the
 * caller; inputs are copied into it, the verifier (algorithm 0 = SpecInfer, 1 = Traversal) runs
 * on `stream`, the five required outputs are copied back and the stream is synchronised before
 * the call returns -- this is the one entry point that synchronises.  Optional outputs and
 * temperature_per_seq are not available here (SPEC_ERR_UNSUPPORTED when set).
 */
int32_t spec_host_staging_bytes(const SpecIn *in, int64_t *bytes);
int32_t spec_verify_host(const SpecIn *in, const SpecOut *out, int32_t algorithm, void *dev_buf,
                         int64_t dev_bytes, void *stream);

/* Launch plan chosen for a vocabulary size and dtype (host-only query, for benchmarks and tests):
 * CTAs per cluster, tokens per CTA slice, dynamic shared memory bytes per CTA, threads per CTA. */
int32_t spec_query_plan(int32_t V, int32_t logits_dtype, int32_t *cluster_size, int32_t *slice_len,
                        int32_t *smem_bytes, int32_t *threads);

/* Number of kernels this library has enqueued in the calling process so far (host-only counter, for
 * benchmarks that report how many launches a timed region made).  Never fails. */
int64_t spec_kernel_launches(void);

/*
 * Test hooks (no counterpart in the paper; not for production callers).  Every wait inside the kernels
 * is bounded (Section "General rules": a wait that runs out is reported as SPEC_DEV_TIMEOUT, nothing
 * hangs); these two settings let a test watch that happen.  wait_cycles: the limit of every on-device
 * wait in clock cycles (<= 0: the default, about 2 s).  hold_slot: index b * N + node of one node whose
 * Traversal weight the every-node kernel then never publishes, so that the node's own wait runs out
 * (-1: none).  Synchronous (copies to constant memory of the current device); call it between
 * verification calls, never while one is in flight.
 */
int32_t spec_test_hooks(int64_t wait_cycles, int32_t hold_slot);

#ifdef __cplusplus
}
#endif
#endif /* SPECVERIFY_H */
