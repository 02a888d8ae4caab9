/*
 * gsd.h - C ABI of the B200 (sm_100a) verification kernels for Graph-structured
 * Speculative Decoding (GSD).
 *
 * The verification stage scores every drafted token of a token graph in ONE pass of the
 * target model and adopts the longest hypothesis the model agrees with (Sec. 1; Sec. 3,
 * single-pass verification; Sec. 4.1, tree attention and longest-path selection;
 * Sec. 5.3-5.4, the merged token graph).  This library provides the two data-parallel
 * parts of that stage for one attention layer / one LM-head output:
 *
 *   gsd_verify_attn  attention of all draft nodes over the committed prefix (KV cache,
 *                    Sec. 4.2) plus exactly the draft nodes named by a per-node ancestor
 *                    bitmask (a flattened token may attend only to its ancestors, Sec. 4.1)
 *   gsd_accept       greedy (deterministic) verification, Sec. 3: per-node vocabulary
 *                    argmax, then the longest accepted root path through the DAG
 *
 * Conventions
 *  - All tensors are dense, row-major, innermost dimension last.  "device" pointers are
 *    CUDA global memory of the current device; "host" pointers are ordinary host memory.
 *  - bf16 tensors are passed as const void* / void* (2-byte elements, IEEE bfloat16).
 *  - Nothing is allocated, freed or synchronised by the device-pointer calls: every
 *    buffer including the workspace is owned by the caller, all work is enqueued on
 *    `stream`, outputs are valid once the stream reaches that point.
 *  - Return value: GSD_OK (0) or a negative gsd_status.  When a host-side check fails
 *    nothing is launched.  Problems only the device can see (malformed CSR, token out of
 *    range, output capacity exceeded, a bounded wait that expired) never trap: the kernel
 *    ORs a GSD_DEV_* bit into *status (if given) and finishes cleanly.
 *  - `stream` is a cudaStream_t passed as void* so that this header needs no CUDA header.
 */
#ifndef GSD_H_
#define GSD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GSD_VERSION 101

typedef enum gsd_status {
    GSD_OK = 0,
    GSD_ERR_NULL_POINTER = -1,   /* a required pointer is NULL */
    GSD_ERR_BAD_SHAPE = -2,      /* unsupported or inconsistent sizes */
    GSD_ERR_MISALIGNED = -3,     /* a tensor base is not sufficiently aligned */
    GSD_ERR_WORKSPACE = -4,      /* workspace missing or too small */
    GSD_ERR_CUDA = -5,           /* a CUDA runtime/driver call failed (see gsd_last_cuda_error) */
    GSD_ERR_UNSUPPORTED = -6     /* requested kernel variant cannot run this shape */
} gsd_status;

/* bits OR-ed into the device status word */
#define GSD_DEV_BAD_CSR      0x1u  /* a parent index outside [0, child) or a bad row pointer; the edge is ignored */
#define GSD_DEV_BAD_TOKEN    0x2u  /* a draft token outside [0, V) (still compared as is) */
#define GSD_DEV_TCAP         0x4u  /* accepted_len exceeded Tcap; the token list was truncated */
#define GSD_DEV_WAIT_EXPIRED 0x8u  /* a bounded in-kernel wait gave up; the output is not valid */
#define GSD_DEV_BAD_SEQ_LEN  0x10u /* seq_lens[b] outside [0, Lmax]; it was clamped */
#define GSD_DEV_CACHE_FULL   0x20u /* gsd_commit_kv: the accepted rows did not all fit below Lmax; the rest was dropped */
#define GSD_DEV_BAD_LOGITS   0x40u /* gsd_accept_sampled, gsd_draft_expand: a logits row without a finite entry (fewer than k for the draft step), or with +inf or NaN */
#define GSD_DEV_DRAFT_FULL   0x80u /* gsd_draft_expand: the node capacity was reached; the remaining children were not created */
#define GSD_DEV_BAD_FRONTIER 0x100u /* gsd_draft_expand: frontier_len, num_nodes or a frontier node id out of range */

#define GSD_DEV_TREE_FULL    0x200u /* gsd_unmerge_tree: the tree capacity was reached; the rest of the level order was dropped */

#define GSD_DEV_BOUNDS       0x400u /* checking build (libgsd_check.so) only: a kernel formed an index outside its tensor; the access was skipped */

#define GSD_MAX_NODES 512          /* largest supported N (draft nodes per sequence) */

/* kernel selection for gsd_verify_attn */
/* GSD_ATTN_AUTO takes the tcgen05 kernel when it supports the shape and the stacked rows of one
 * (sequence, kv head), N * Hq/Hkv, number at least 64; everything else runs on the mma.sync
 * kernel, which reaches roughly a sixth of the tensor throughput (group sizes 3, 6, 12, ... and
 * D == 64 therefore stay correct but slow).  Asking for GSD_ATTN_TCGEN05 on a shape it does
 * not support returns GSD_ERR_UNSUPPORTED. */
#define GSD_ATTN_SPLIT_BALANCED (-1)      /* values of gsd_attn_params.num_splits */
#define GSD_ATTN_SPLIT_PER_SEQUENCE (-2)

#define GSD_ATTN_AUTO 0
#define GSD_ATTN_MMA  1            /* warp-level mma.sync kernel: D in {64,128}, any N, any group size */
#define GSD_ATTN_TCGEN05 2         /* tcgen05/TMEM/TMA kernel: D == 128 and Hq/Hkv a divisor of 128 */

typedef struct gsd_attn_params {
    int32_t B;            /* sequences */
    int32_t N;            /* draft nodes per sequence, 1..GSD_MAX_NODES; node 0 is the root */
    int32_t Hq;           /* query heads */
    int32_t Hkv;          /* key/value heads; Hq % Hkv == 0; q-head h uses kv-head h / (Hq/Hkv) */
    int32_t D;            /* head dimension: 64 or 128 */
    int32_t Lmax;         /* padded cache length (rows per sequence in k_cache/v_cache), >= 1 */
    float softmax_scale;  /* <= 0 selects 1/sqrt(D) */
    int32_t num_splits;   /* key-range splits per (sequence, kv head, row tile); 0 = choose;
                             GSD_ATTN_SPLIT_BALANCED = equal shares of key tiles per CTA, dealt out on the
                             device from seq_lens; GSD_ATTN_SPLIT_PER_SEQUENCE = a split count per sequence,
                             chosen on the device from seq_lens so that all units are about equally long
                             (both: tcgen05 kernel; the mma.sync kernel reads them as 0) */
    int32_t kernel;       /* GSD_ATTN_AUTO / _MMA / _TCGEN05 */
} gsd_attn_params;

typedef struct gsd_accept_params {
    int32_t B;     /* sequences */
    int32_t N;     /* draft nodes per sequence, 1..GSD_MAX_NODES */
    int32_t V;     /* vocabulary size, >= 1 */
    int32_t Ecap;  /* row length of parent_idx, >= 1 */
    int32_t Tcap;  /* row length of accepted_tokens / accepted_nodes, >= 1 (N always suffices) */
} gsd_accept_params;

int gsd_version(void);
const char* gsd_status_string(int status);
/* Text of the last CUDA error this library saw on the calling thread ("" if none). */
const char* gsd_last_cuda_error(void);

/*
 * gsd_verify_attn - DAG-masked attention of the draft nodes (Sec. 4.1 tree attention over
 * the flattened token graph, Sec. 4.2 KV cache).
 *
 * For every sequence b, node n and query head h (kv head c = h / (Hq/Hkv)):
 *   keys   = cache rows j < seq_lens[b]  plus  draft rows j with bit j of ancestor_mask[b][n] set
 *   out[b,n,h,:] = sum_j softmax_j(scale * <q[b,n,h,:], K_j[c,:]>) * V_j[c,:]
 * bf16 inputs, fp32 accumulation, bf16 output (round to nearest even).  Mask bits are
 * honoured literally (no implicit diagonal, no triangularity assumed); bits >= N are
 * ignored.  Cache rows at positions >= seq_lens[b] never reach the result, whatever
 * they contain.  A row with no visible key yields zeros.
 *
 *   q              [B, N, Hq, D]      bf16  device  in
 *   k_cache        [B, Lmax, Hkv, D]  bf16  device  in
 *   v_cache        [B, Lmax, Hkv, D]  bf16  device  in
 *   draft_k        [B, N, Hkv, D]     bf16  device  in
 *   draft_v        [B, N, Hkv, D]     bf16  device  in
 *   ancestor_mask  [B, N, W] uint32, W = ceil(N/32), device, in; bit j of a row is
 *                  word j / 32, bit j % 32
 *   seq_lens       [B] int32 device in; 0 <= seq_lens[b] <= Lmax (clamped and flagged otherwise)
 *   out            [B, N, Hq, D]      bf16  device  out
 *   p              host
 *   workspace      device scratch of at least gsd_verify_attn_workspace_bytes(p) bytes,
 *                  256-byte aligned; may be NULL when that size is 0.  Contents are
 *                  undefined before and after the call.
 *   status         device int32 word or NULL; GSD_DEV_* bits are OR-ed in (never cleared)
 *   stream         cudaStream_t
 *
 * All tensor bases must be 16-byte aligned.  Calls that share a workspace must not
 * overlap on the device.  Errors: see gsd_status; nothing is launched on a host error.
 */
int gsd_verify_attn(const void* q, const void* k_cache, const void* v_cache,
                    const void* draft_k, const void* draft_v, const uint32_t* ancestor_mask,
                    const int32_t* seq_lens, void* out, const gsd_attn_params* p,
                    void* workspace, size_t workspace_bytes, int32_t* status, void* stream);

/*
 * gsd_debug_attn_wait - test hook for the bounded waits of the tcgen05 back end of
 * gsd_verify_attn (no counterpart in the paper).  Every in-kernel wait (on a copy, on a tensor
 * core result, on another warp) gives up after a time limit, 2 s by default: the kernel then ORs
 * GSD_DEV_WAIT_EXPIRED into *status, all its warps leave their loops, copies and tensor-core
 * work already under way are awaited (again with the limit), the tensor memory is released and
 * the launch ends normally; `out` is not valid, the next call works as usual.
 *   limit_ns          new limit for later launches of this process (0 = back to the default)
 *   withhold_first_k  non-zero: every CTA of later launches announces but never issues the copy of
 *                     its first key tile, so that a wait really runs out - for tests of the path
 *                     above; zero switches it off again
 */
void gsd_debug_attn_wait(uint64_t limit_ns, int32_t withhold_first_k);

/* Bytes of workspace gsd_verify_attn needs for *p on the current device (0 on invalid
 * parameters or when none is needed). */
size_t gsd_verify_attn_workspace_bytes(const gsd_attn_params* p);

/* The number of key-range splits gsd_verify_attn would use for *p on the current device
 * (p->num_splits if positive, else the automatic choice); GSD_ATTN_SPLIT_BALANCED or
 * GSD_ATTN_SPLIT_PER_SEQUENCE when the work is shared out on the device; 0 on invalid parameters. */
int gsd_verify_attn_num_splits(const gsd_attn_params* p);

/*
 * gsd_accept - deterministic verification and longest-path selection (Sec. 3: a drafted
 * token is accepted only if the target model would generate the same token; after a
 * rejection the rest of the hypothesis is dropped and the target model supplies the next
 * token.  Sec. 4.1 / Sec. 1: the longest hypothesis from the root is adopted).
 *
 *   a[b,n] = lowest index i with logits[b,n,i] equal to the row maximum over non-NaN
 *            entries (0 if the row is all NaN)
 *   edge p->v is accepted iff draft_tokens[b,v] == a[b,p]
 *   the chosen path v0=0,v1..vm is the longest root path of accepted edges; among equally
 *   long ones the lowest end node, then step by step the lowest predecessor that carries
 *   length-1
 *   accepted_tokens[b,:] = tok[v1..vm], a[b,vm], then -1 padding;  accepted_len[b] = m+1
 *
 *   logits          [B, N, V] fp32 device in
 *   draft_tokens    [B, N] int32 device in; node 0 is the root (its token is not emitted)
 *   parent_ptr      [B, N+1] int32 device in; CSR row pointers, local to sequence b
 *   parent_idx      [B, Ecap] int32 device in; parents of v are idx[ptr[v] .. ptr[v+1]);
 *                   every parent index must be < v (topological numbering)
 *   accepted_tokens [B, Tcap] int32 device out
 *   accepted_len    [B] int32 device out
 *   accepted_nodes  [B, Tcap] int32 device out or NULL: v0..vm then -1 padding
 *   p               host
 *   workspace       device scratch >= gsd_accept_workspace_bytes(p), 8-byte aligned
 *   status          device int32 word or NULL
 *   stream          cudaStream_t
 *
 * logits must be 4-byte aligned; 16-byte alignment with V % 4 == 0 enables vector loads.
 */
int gsd_accept(const float* logits, const int32_t* draft_tokens, const int32_t* parent_ptr,
               const int32_t* parent_idx, int32_t* accepted_tokens, int32_t* accepted_len,
               int32_t* accepted_nodes, const gsd_accept_params* p, void* workspace,
               size_t workspace_bytes, int32_t* status, void* stream);

size_t gsd_accept_workspace_bytes(const gsd_accept_params* p);

/*
 * gsd_accept_sampled - non-deterministic verification of the token graph (Sec. 3: a drafted
 * token is accepted with probability min(1, p/q); the first rejection discards the rest of the
 * hypothesis and the target model regenerates that token; Sec. 6.4 runs this on the graph;
 * longest-path selection as in Sec. 4.1).  The random numbers are inputs, so the call is a pure
 * function.  Readings (the paper gives the rule for a single hypothesis only):
 *   - the test is applied to every step parent -> v of the graph, with p the target
 *     probability softmax(logits[b][parent])[draft_tokens[b][v]] and q = draft_q[b][v]:
 *         accepted  iff  u_accept[b][v] * q < p        (u < min(1, p/q); q = 0 accepts iff p > 0)
 *   - the hypothesis is the longest root path all of whose steps are accepted; ties as in
 *     gsd_accept (lowest end node, then lowest predecessor walking back);
 *   - the regenerated token follows the sampling scheme that Sec. 3 cites, which is what makes
 *     the accepted tokens follow the target model's distribution: with P = softmax(logits[b][end
 *     node]) and Q = softmax(draft_logits[b][end node]) it is drawn from the residual
 *     max(0, P_j - Q_j) / sum_i max(0, P_i - Q_i) when the end node has a child in the graph (its
 *     drafted continuations were all rejected; several rejected siblings share the one
 *     residual), and from P itself when the end node has no child, when the residual has no
 *     mass (sum <= 1e-6) or when draft_logits is NULL.  The draw inverts the cumulative weights
 *     in index order: the smallest t with sum_{j<=t} w_j > u_sample[b] * sum_j w_j (the last t
 *     with w_t > 0 if rounding leaves none).
 * Temperature / nucleus filtering are the caller's: pass logits already divided by the
 * temperature (and with filtered entries at -inf).
 *
 *   logits, draft_tokens, parent_ptr, parent_idx   device, as for gsd_accept; every logits row
 *                    must hold at least one finite value, no +inf and no NaN (GSD_DEV_BAD_LOGITS)
 *   draft_logits     device const f32 [B,N,V] or NULL: the draft model's logits at every node (the
 *                    distribution the node's children were drafted from); only the row of the end
 *                    node of each sequence is read.  NULL: the regenerated token is always drawn
 *                    from P (no residual)
 *   draft_q          device const f32 [B,N]: the probability the draft model gave node v's token
 *                    when it drafted it (entry 0, the root, is not read)
 *   u_accept         device const f32 [B,N]: one number in [0,1) per node (entry 0 not read)
 *   u_sample         device const f32 [B]: one number in [0,1) per sequence
 *   accepted_tokens, accepted_len, accepted_nodes   device outputs as for gsd_accept; the entry
 *                    after the drafted tokens of the path is the regenerated token
 *   workspace        device scratch of gsd_accept_sampled_workspace_bytes(p) bytes, 8-byte
 *                    aligned, arbitrary contents; the call clears what has to start at zero
 * The softmax statistics are accumulated in fp32 (ex2.approx); a step whose two sides differ by
 * less than a few 1e-6 relative may be decided differently from an exact evaluation.
 * Errors and status bits as for gsd_accept, plus GSD_DEV_BAD_LOGITS.  Asynchronous on `stream`.
 */
size_t gsd_accept_sampled_workspace_bytes(const gsd_accept_params* p);
int gsd_accept_sampled(const float* logits, const int32_t* draft_tokens, const int32_t* parent_ptr,
                       const int32_t* parent_idx, const float* draft_logits, const float* draft_q,
                       const float* u_accept, const float* u_sample, int32_t* accepted_tokens,
                       int32_t* accepted_len,
                       int32_t* accepted_nodes, const gsd_accept_params* p, void* workspace,
                       size_t workspace_bytes, int32_t* status, void* stream);

/*
 * gsd_draft_expand - one growth step of the draft token graph on the device (Sec. 4: token
 * tree of out-degree k; Sec. 4.2: probability pruning and sibling pruning; Sec. 5.2:
 * tau-redundant nodes; Sec. 5.3: merging).  For every sequence b the frontier nodes
 * frontier[b][0..frontier_len[b]) are expanded in order.  For a frontier node p with draft
 * distribution P = softmax(logits[b][fi]):
 *   - its k children are the k most probable tokens, best first, ties to the lowest token id;
 *     they become the nodes num_nodes[b], num_nodes[b]+1, ... with tokens[c] = token,
 *     tree_parent[c] = p, prob[c] = the token's probability q, merge_to[c] = -1;
 *   - leaf[c] = 1 if q < theta_prob (probability pruning) or q < theta_sib * q_best with q_best
 *     the largest of the k sibling probabilities (sibling pruning); pruned children are kept as
 *     leaves, as the paper marks them;
 *   - a child is tau-redundant if the tau tokens that end at it along its tree path (itself and
 *     tau - 1 tree ancestors; a shorter path does not count) equal the tau tokens ending at a
 *     node with a lower id (of this or an earlier step): then leaf[c] = 1 and merge_to[c] = the
 *     lowest such id, the first occurrence (whose successors verification re-uses, Sec. 5.3).
 * new_frontier[b] lists the new nodes that are not leaves, in id order.  Readings: the root's
 * token is part of the paths; the first occurrence may itself be a pruned leaf; the merge edges
 * are reported (merge_to), the verification DAG's parent lists are the caller's to derive:
 * parents(x) = { tree_parent[x] } + { r : merge_to[r] == tree_parent[x] }.
 *
 *   logits        device const f32 [B,F,V], draft-model logits of the frontier nodes (rows at or
 *                 past frontier_len[b] are not read); every row needs at least k entries above
 *                 -inf, no +inf, no NaN (else GSD_DEV_BAD_LOGITS)
 *   frontier      device const i32 [B,F] node ids < num_nodes[b];  frontier_len  device const i32 [B]
 *   tokens, tree_parent, merge_to   device i32 [B,Ncap];  leaf  device u8 [B,Ncap];
 *   prob          device f32 [B,Ncap];  num_nodes  device i32 [B]   - the graph, updated in place
 *                 (node 0 is the root: tree_parent -1); Ncap <= GSD_MAX_NODES; when the capacity
 *                 is reached the remaining children are dropped (GSD_DEV_DRAFT_FULL)
 *   new_frontier  device i32 [B,F*k] (only the first new_frontier_len[b] entries are written);
 *   new_frontier_len  device i32 [B]
 *   workspace     device scratch of gsd_draft_expand_workspace_bytes(p) bytes, 8-byte aligned,
 *                 arbitrary contents
 * The probabilities are fp32 (ex2.approx); a pruning comparison whose two sides differ by less
 * than a few 1e-6 relative may fall either way.  The order of the children never depends on
 * arithmetic (it compares logits).  1 <= k <= GSD_DRAFT_MAX_K, k <= V, tau >= 1.
 * Returns GSD_OK or a negative gsd_status; asynchronous on `stream`; allocates nothing.
 */
#define GSD_DRAFT_MAX_K 8
typedef struct gsd_draft_params {
    int32_t B, F, V, Ncap, k, tau;
    float theta_prob, theta_sib;
} gsd_draft_params;
size_t gsd_draft_expand_workspace_bytes(const gsd_draft_params* p);
int gsd_draft_expand(const float* logits, const int32_t* frontier, const int32_t* frontier_len,
                     int32_t* tokens, int32_t* tree_parent, int32_t* merge_to, uint8_t* leaf,
                     float* prob, int32_t* num_nodes, int32_t* new_frontier,
                     int32_t* new_frontier_len, const gsd_draft_params* p, void* workspace,
                     size_t workspace_bytes, int32_t* status, void* stream);

/*
 * gsd_accept_static - gsd_accept without a workspace argument.  (The paper has no counterpart
 * for this call; it is a packaging variant of gsd_accept.)
 *
 * Some callers have no device memory to give: a plug-in running inside a serving process
 * whose host application has already claimed the GPU's memory for its own pool, a caller
 * that is handed tensors by another runtime and has no allocator of its own, or code on a
 * latency-critical path where cudaMalloc (which may synchronise the whole device) is off
 * limits.  For them the scratch that gsd_accept needs (8 bytes per draft node + 4 bytes per
 * sequence) lives in a fixed array inside the library image, GSD_STATIC_SCRATCH_BYTES long;
 * every GPU on which the library is used holds that array until the process exits.
 *
 * Same arguments, results, status bits and error codes as gsd_accept, minus workspace and
 * workspace_bytes.  Limit: B * N <= GSD_STATIC_MAX_ROWS; larger problems are refused with
 * GSD_ERR_WORKSPACE (and a text in gsd_last_cuda_error) before anything is launched.
 * The call allocates and frees nothing.
 *
 * The first call on each device looks up the array's device address (the device must be
 * current, as for every call here); make that first call outside any stream capture.
 * All calls on a device share the one array: it keeps whatever the last call left in it, the
 * part a call uses is cleared on `stream` before its kernel touches it, and two calls that can
 * overlap on the GPU (different streams, no dependency) race on it - serialise them.
 */
#define GSD_STATIC_MAX_ROWS 16384
#define GSD_STATIC_SCRATCH_BYTES (GSD_STATIC_MAX_ROWS * 8 + GSD_STATIC_MAX_ROWS * 4 + 256)
int gsd_accept_static(const float* logits, const int32_t* draft_tokens, const int32_t* parent_ptr,
                      const int32_t* parent_idx, int32_t* accepted_tokens, int32_t* accepted_len,
                      int32_t* accepted_nodes, const gsd_accept_params* p, int32_t* status,
                      void* stream);

/*
 * gsd_build_mask - the ancestor bitmask that gsd_verify_attn takes, built on the device from
 * the parent lists (tree attention lets a token attend only to its ancestors, Sec. 4.1; in
 * the merged token graph of Sec. 5.3 a node has several parents and sees the union of their
 * ancestors).
 *
 *   ancestor_mask[b][n] has bit j (word j / 32, bit j % 32) set iff j == n or node n can be
 *   reached from node j along parent edges; bits >= N are zero.
 *
 *   parent_ptr     [B, N+1] int32 device in   (CSR row pointers, local to the sequence)
 *   parent_idx     [B, Ecap] int32 device in  (every parent index must be < its child)
 *   ancestor_mask  [B, N, ceil(N/32)] uint32 device out
 *   status         device int32 word or NULL (GSD_DEV_BAD_CSR: an edge or row pointer was ignored)
 *   stream         cudaStream_t
 *
 * N <= GSD_MAX_NODES.  No workspace, no allocation, asynchronous on `stream`.
 */
int gsd_build_mask(const int32_t* parent_ptr, const int32_t* parent_idx, uint32_t* ancestor_mask,
                   int32_t B, int32_t N, int32_t Ecap, int32_t* status, void* stream);

/*
 * gsd_unmerge_tree - the token graph reverted to a tree for verification (Sec. 5.4, Fig. 4: before
 * verification the merged nodes are "unmerged": the successors of a redundant node are replicated
 * from the node it was merged into, and the tree is verified as in tree-structured decoding).
 * On the verification DAG, given by parent lists, this is its unfolding from the root: one tree
 * node per root path.  The tree can then be fed to gsd_build_mask / gsd_verify_attn / gsd_accept
 * (gather q, draft K/V and logits rows by tree_source) as an alternative to verifying the DAG
 * directly.
 *
 *   tree node 0 is the root.  Tree nodes are numbered level by level, inside a level by (tree
 *   index of the parent, then id of the copied DAG node), so a parent precedes its children.
 *   Nodes deeper than max_depth edges below the root are not created (a merge pattern that
 *   repeats along one path could otherwise unfold without end); when Ucap nodes exist the rest
 *   of the level order is dropped (GSD_DEV_TREE_FULL).
 *
 *   draft_tokens  [B, N] int32 device in      parent_ptr [B, N+1], parent_idx [B, Ecap] int32
 *                 device in, as for gsd_accept (at most GSD_UNMERGE_MAX_EDGES edges per sequence
 *                 are read; a parent listed twice in one row counts once)
 *   tree_tokens, tree_parent, tree_source  [B, Ucap] int32 device out: token, tree index of the
 *                 parent (-1 for the root) and copied DAG node of every tree node; -1 past the end
 *   tree_count    [B] int32 device out: tree nodes created
 *   status        device int32 word or NULL (GSD_DEV_BAD_CSR, GSD_DEV_TREE_FULL);  stream: cudaStream_t
 *
 * N <= GSD_MAX_NODES.  No workspace, no allocation, asynchronous on `stream`.
 */
#define GSD_UNMERGE_MAX_EDGES 4096
int gsd_unmerge_tree(const int32_t* draft_tokens, const int32_t* parent_ptr, const int32_t* parent_idx,
                     int32_t* tree_tokens, int32_t* tree_parent, int32_t* tree_source, int32_t* tree_count,
                     int32_t B, int32_t N, int32_t Ecap, int32_t Ucap, int32_t max_depth, int32_t* status,
                     void* stream);

typedef struct gsd_commit_params {
    int32_t B;     /* sequences */
    int32_t N;     /* draft nodes per sequence */
    int32_t Hkv;   /* key/value heads */
    int32_t D;     /* head dimension, a multiple of 8 */
    int32_t Lmax;  /* rows per sequence in k_cache / v_cache */
    int32_t Tcap;  /* row length of accepted_nodes */
} gsd_commit_params;

/*
 * gsd_commit_kv - make the accepted path part of the committed context: the KV-cache update
 * that follows verification (the paper counts the cache update under "Others" in its time
 * breakdown, Sec. 7.1 / Table 3; KV caching, Sec. 4.2).
 *
 * For every sequence b, with len = min(accepted_len[b], Tcap) and the path nodes
 * accepted_nodes[b][0..len) (node 0, the root whose K/V were not yet cached, then the accepted
 * draft nodes), the draft_k / draft_v rows of those nodes are copied to cache positions
 * seq_lens[b], seq_lens[b]+1, ... and seq_lens[b] is advanced by the number of rows written.
 * Rows that would land at or past Lmax are dropped (GSD_DEV_CACHE_FULL); node ids outside
 * [0, N) are skipped (GSD_DEV_BAD_CSR).  Nothing else in the cache is touched.
 *
 *   k_cache, v_cache  [B, Lmax, Hkv, D] bf16 device in/out
 *   draft_k, draft_v  [B, N, Hkv, D]    bf16 device in
 *   accepted_nodes    [B, Tcap] int32 device in   (as written by gsd_accept)
 *   accepted_len      [B]       int32 device in
 *   seq_lens          [B]       int32 device in/out
 *   status            device int32 word or NULL;  stream: cudaStream_t
 *
 * Tensor bases 16-byte aligned.  No workspace, no allocation, asynchronous on `stream`.
 */
int gsd_commit_kv(void* k_cache, void* v_cache, const void* draft_k, const void* draft_v,
                  const int32_t* accepted_nodes, const int32_t* accepted_len, int32_t* seq_lens,
                  const gsd_commit_params* p, int32_t* status, void* stream);

/*
 * gsd_verify_step_host - one whole verification step from HOST buffers: copies every
 * input to the device arena, runs gsd_verify_attn and gsd_accept, copies `out`,
 * accepted_tokens, accepted_len (and accepted_nodes if non-NULL) back and waits for the
 * stream.  Same operations and passages as the two calls above; this entry point exists
 * for callers that keep their tensors in host memory and to measure the step end to end.
 *
 * All tensor pointers are host pointers with the layouts given above (pinned memory makes
 * the copies asynchronous and faster, pageable memory works too).  `arena` is a device
 * buffer of at least gsd_verify_step_host_arena_bytes(ap, cp) bytes, 256-byte aligned,
 * owned by the caller.  `device_status_out` (host, may be NULL) receives the device
 * status word of this step.  ap->B == cp->B and ap->N == cp->N are required.
 *
 * The inputs travel on a copy stream that the library creates at the first call on a device
 * (with three events; all kept until the process exits), the attention inputs first: the
 * attention runs on `stream` as soon as they have landed, and its output goes back to the host
 * while the logits are still coming in.  The copy stream waits for the work already queued on
 * `stream`, and the call returns after `stream` has drained, so the arena may be reused at once.
 * Calls on one device must not be made from several host threads at the same time.
 */
int gsd_verify_step_host(const void* q, const void* k_cache, const void* v_cache,
                         const void* draft_k, const void* draft_v,
                         const uint32_t* ancestor_mask, const int32_t* seq_lens, void* out,
                         const gsd_attn_params* ap, const float* logits,
                         const int32_t* draft_tokens, const int32_t* parent_ptr,
                         const int32_t* parent_idx, int32_t* accepted_tokens,
                         int32_t* accepted_len, int32_t* accepted_nodes,
                         const gsd_accept_params* cp, void* arena, size_t arena_bytes,
                         int32_t* device_status_out, void* stream);

size_t gsd_verify_step_host_arena_bytes(const gsd_attn_params* ap, const gsd_accept_params* cp);

#ifdef __cplusplus
}
#endif
#endif /* GSD_H_ */
