/*
 * rtma.h -- C ABI of the RandomTMA / SuperTMA data-parallel hot path on one
 * NVIDIA B200 (sm_100a).
 *
 * "TMA" is the paper's Time-based Model Aggregation (Sec. 3.1), not the GPU's
 * tensor-memory unit.  The calls follow the paper's problem statement (Sec. 3,
 * requirements R1 and R2): a partition function alpha that maps nodes to the M
 * trainers, the node-induced subgraph of every part, independent local training
 * on each part (Algorithm 2), and the aggregation of the trainers' parameters
 * (Algorithm 1).
 *
 * Conventions
 *  - Every function returns an int32_t status: RTMA_OK (0) or a negative
 *    RTMA_ERR_* code.  Nothing throws or aborts across this boundary;
 *    rtma_last_error(ctx) gives the text of the last failure on that context.
 *  - Unless a parameter says "host", every array pointer is a DEVICE pointer to
 *    memory that the caller allocated and owns (for instance the data pointer
 *    of a torch tensor).  The library never frees it and keeps no reference to
 *    it after the call returns.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *    stream).  Calls only enqueue work on it and return without synchronising,
 *    except where stated.  Outputs are valid once the stream has drained.
 *  - The context owns one scratch arena on its device; it grows (cudaMalloc +
 *    cudaFree, which synchronise the device) only when a call needs more than
 *    any call before it.  Every call on a context uses that scratch, so calls on
 *    one context must be ordered: the same stream, or the earlier call's stream
 *    drained first.  The one case the library orders itself: after a local-training
 *    call that spread its trainers over several streams, the next call on the context
 *    (on whatever stream) first waits, on the device, for all of those streams.  A
 *    context must not be used from two host threads at the same time.
 *  - Node ids and column indices are int32; row offsets are int32 or int64 on
 *    input and int64 on output.  At most RTMA_MAX_PARTS trainers.
 */
#ifndef RTMA_H_
#define RTMA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define RTMA_MAX_PARTS 64
#define RTMA_MAX_LAYERS 8

enum {
    RTMA_OK = 0,
    RTMA_ERR_INVALID_ARG = -1, /* null pointer, negative size, M out of range ...        */
    RTMA_ERR_UNSUPPORTED = -2, /* a shape or mode this build does not implement           */
    RTMA_ERR_WORKSPACE = -3,   /* the scratch arena cannot be made large enough           */
    RTMA_ERR_OVERFLOW = -4,    /* a count does not fit the index type of its output       */
    RTMA_ERR_CUDA = -5,        /* a CUDA runtime call failed; text in rtma_last_error     */
    RTMA_ERR_TIMEOUT = -6,     /* a bounded device-side wait ran out (kernel gave up)     */
    RTMA_ERR_BOUNDS = -7       /* checked build only: an index in the caller's data was out of range */
};

typedef struct rtma_ctx rtma_ctx;

/* Creates a context on CUDA device `device` and reserves `workspace_bytes` of scratch
 * (0 = reserve lazily).  Synchronous.  *out is NULL on failure.                          */
int32_t rtma_create(rtma_ctx** out, int32_t device, size_t workspace_bytes);
/* Synchronises the device, frees the scratch arena and the context.                      */
int32_t rtma_destroy(rtma_ctx* ctx);
/* Text of the last error on this context ("" if none).  Owned by the context.            */
const char* rtma_last_error(const rtma_ctx* ctx);
/* Synchronises the device and reports RTMA_ERR_TIMEOUT if any kernel launched through this
 * context since the last check gave up on one of its bounded device-side waits (the
 * tensor-core kernels wait on mbarriers with an iteration limit instead of spinning for
 * ever), RTMA_ERR_INVALID_ARG if a local-training call since the last check was given a
 * subgraph that is not symmetric; RTMA_OK otherwise.  rtma_train_host calls it before
 * returning.  In the checked build of the library (compiled with -DRTMA_BOUNDS; every index taken
 * from the caller's data is range-checked and an offending access is skipped, not made) it
 * also reports RTMA_ERR_BOUNDS with the first offending index.                               */
int32_t rtma_check(rtma_ctx* ctx);
/* 1 if this library is the checked build (-DRTMA_BOUNDS), else 0.                           */
int32_t rtma_bounds_checked(void);
/* Bytes of scratch currently held by the context.                                        */
size_t rtma_workspace_bytes(const rtma_ctx* ctx);
/* Caps the scratch arena at `bytes` (0 = no cap, the default): no later call grows it beyond
 * that, and a call that cannot work inside it returns RTMA_ERR_WORKSPACE.  An arena that is
 * already larger is kept but only its first `bytes` are used by rtma_local_steps, which then
 * runs the trainers of a stream in successive waves, each wave re-using the same scratch; the
 * results are bit for bit those of a single wave.  For hosts that share the GPU with other
 * tenants of a fixed memory budget.  The paper has no counterpart.                          */
int32_t rtma_set_workspace_limit(rtma_ctx* ctx, size_t bytes);
/* How rtma_local_steps forms the mean aggregation Abar H (Theorem 2) and its transpose for a part:
 *   0  always by gathering the neighbours' rows;
 *   1  (default) per part: where at least half of the entries of a sample of its rows (every 64th)
 *      have their column within 128 rows of the row's 128-row tile, and those rows have 4 entries or
 *      more on average - the nodes of a super-node stored together (Sec. 3.2, rows ordered by
 *      super-node as rtma_partition_grouped leaves them) - the entries inside that window are taken
 *      from dense tiles on the tensor cores and only the others are gathered;
 *   2  the tensor-core tiles for every part (for tests).
 * The decision depends on the part alone, so a trainer's results do not depend on which other
 * trainers share its call; a part in which some row repeats an entry inside that window always
 * gathers.  GCN layers, and rows of fewer than 16 values, always gather.  In modes 1 and 2 the
 * training calls wait once per wave, while they set up, for the stream to deliver the per-part
 * decision (twice where some part takes the tiles); in mode 0 they only enqueue.
 * Returns RTMA_ERR_INVALID_ARG for any other mode.                                           */
int32_t rtma_set_dense_aggregation(rtma_ctx* ctx, int32_t mode);

/* ---- R1: partition function (Sec. 3.2.2, RandomTMA and SuperTMA) -----------------------
 * part_id[v] = h(seed XOR g(v)) mod M, where h is one step of the SplitMix64 generator and
 * g(v) = v when group_id is NULL (RandomTMA: every node assigned independently) or
 * g(v) = group_id[v] (SuperTMA: every super-node / mini-cluster assigned as a whole; ids
 * need not be dense).  Also produces the ordered member lists alpha^{-1}(i) of the
 * Preliminaries: part_offsets[M+1] (exclusive scan of part sizes), perm[n] (global ids
 * sorted by (part, id)), local_id[n] (rank of v inside its part).
 * 1 <= M <= RTMA_MAX_PARTS, 0 <= n < 2^31.  All four outputs are always written.          */
int32_t rtma_partition(rtma_ctx* ctx, int64_t n, const int32_t* group_id, uint64_t seed,
                       int32_t M, int32_t* part_id, int64_t* part_offsets, int32_t* perm,
                       int32_t* local_id, void* stream);

/* The same assignment with every super-node's members adjacent in memory: inside a part the
 * nodes are ordered by super-node id (as a signed 32-bit number), then by node id, instead of
 * by node id alone.  SuperTMA assigns a super-node as a whole (Sec. 3.2.2), so all its members
 * are in the part, and in the graphs the scheme is meant for most of a node's neighbours are in
 * its own super-node (mini-clusters, Sec. 3.2.2): with this order they are nearby rows of the
 * part, which the aggregation kernels of rtma_local_steps turn into cache hits.  part_id and
 * part_offsets equal rtma_partition's; perm and local_id differ only in the order inside each
 * part.  group_id == NULL is rtma_partition.  Arguments, limits and errors as rtma_partition. */
int32_t rtma_partition_grouped(rtma_ctx* ctx, int64_t n, const int32_t* group_id, uint64_t seed,
                               int32_t M, int32_t* part_id, int64_t* part_offsets, int32_t* perm,
                               int32_t* local_id, void* stream);

/* The same partition for callers that must not allocate device memory.  (The paper has no
 * counterpart: this is a deployment variant of rtma_partition.)  Some hosts of this library
 * cannot call cudaMalloc at the point where they partition: code running while a CUDA graph is
 * being captured or inside a memory pool whose size is fixed in advance, services that pin their
 * whole device budget at start-up, and callers holding locks under which an allocation (which may
 * synchronise the device) is forbidden.  rtma_partition takes its scratch from the context's
 * arena, which it may have to grow; this entry point needs no context and takes its scratch from
 * a fixed array compiled into the library (about 3 MB, held on every GPU that loads the library
 * until the process exits).  It calls no cudaMalloc / cudaFree and no allocating routine.
 *   Limit: ceil(n / 1024) * M <= RTMA_PARTITION_STATIC_MAX_CELLS (e.g. 4,194,304 nodes at M = 64,
 *   33,554,432 nodes at M = 8); beyond it the call returns RTMA_ERR_WORKSPACE and does nothing.
 *   Arguments and results are exactly those of rtma_partition (device pointers, same outputs bit
 *   for bit); `device` is the CUDA device the pointers live on and is made current.
 *   The first call on a device looks up the scratch array's device address (cudaGetSymbolAddress);
 *   make that first call before any stream capture begins.
 *   All calls share the one array, which keeps the previous call's contents (nothing in it needs
 *   clearing: every cell is rewritten before it is read).  Two calls whose kernels overlap on the
 *   GPU -- different streams without ordering, or different host threads -- race on it: order them.
 *   Errors: RTMA_ERR_* as elsewhere; rtma_partition_static_error() returns the text of the last
 *   failure of this entry point (one buffer for the process, not thread safe).               */
#define RTMA_PARTITION_STATIC_MAX_CELLS 262144
int32_t rtma_partition_static(int32_t device, int64_t n, const int32_t* group_id, uint64_t seed,
                              int32_t M, int32_t* part_id, int64_t* part_offsets, int32_t* perm,
                              int32_t* local_id, void* stream);
const char* rtma_partition_static_error(void);

/* ---- node-induced subgraphs G^(i) (Preliminaries) --------------------------------------
 * Keeps CSR entry (u,v) iff part_id[u] == part_id[v] and emits, for every part, a CSR over
 * local ids with rows in local order and the input's column order preserved.
 *   rowptr       [n+1], int64 if rowptr_is_64 else int32;  col [rowptr[n]] int32.
 *   rowptr_out   [n+M] int64: part p's n_p+1 zero-based offsets start at part_offsets[p]+p.
 *   edge_offsets [M+1] int64: part p's entries are col_out[edge_offsets[p] .. edge_offsets[p+1]).
 *   kept_cut     [2]   int64: entries kept, entries dropped (kept + cut = rowptr[n]).
 * Two phases.  col_out == NULL: COUNT -- writes rowptr_out, edge_offsets and kept_cut; read
 * edge_offsets[M] back (after draining the stream) to size col_out.  col_out != NULL: FILL --
 * reads rowptr_out and edge_offsets as the count phase left them and writes col_out only.
 * COUNT waits for the stream once (it reads rowptr[n], 8 bytes) and leaves, in a buffer of the
 * context of rowptr[n] / 8 + 4 n bytes (kept until the context is destroyed, not part of the
 * scratch arena), one bit per entry: kept or not.  A FILL that follows the COUNT on the same n, M, rowptr,
 * col and part_id pointers reads those bits and the kept entries only; any other FILL (or one
 * after a COUNT that found no memory for the bits) looks every entry's part up again.  Same
 * result either way.
 * part_id / part_offsets / perm / local_id are rtma_partition's outputs.                  */
int32_t rtma_build_induced_csr(rtma_ctx* ctx, int64_t n, int32_t rowptr_is_64, const void* rowptr,
                               const int32_t* col, int32_t M, const int32_t* part_id,
                               const int64_t* part_offsets, const int32_t* perm,
                               const int32_t* local_id, int64_t* rowptr_out, int32_t* col_out,
                               int64_t* edge_offsets, int64_t* kept_cut, void* stream);

/* dst[i] = src[perm[i]] for rows of row_bytes bytes: brings features and labels into
 * partition order ("load G_train^(i)", Algorithm 2).  src and dst must not overlap.       */
int32_t rtma_gather_rows(rtma_ctx* ctx, int64_t n, int64_t row_bytes, const void* src,
                         const int32_t* perm, void* dst, void* stream);

/* ---- local training (Algorithm 2, the loop body with a plain SGD optimizer) ------------
 * Model: L GraphSAGE-mean layers, Z^l = H^l Ws^l + (Abar H^l) Wn^l + b^l, ReLU between
 * layers, softmax cross-entropy averaged over the part's nodes.  Abar is the part's
 * row-normalised adjacency (Theorem 2): the mean over LOCAL neighbours, zero for a node
 * without any.  dims[0] = feature width, dims[L] = number of classes.
 * Parameters of one trainer: flat float vector of rtma_param_count() entries, layer after
 * layer: Ws[d_l][d_{l+1}], Wn[d_l][d_{l+1}], b[d_{l+1}], all row-major.
 *
 * Variants (Sec. 4.1 "GNN Encoders": GCN or GraphSAGE encoders, PReLU, Layer Normalization
 * before the activation), all zero = the model above:
 *   encoder = 1  GCN layers, Z^l = (Ahat H^l) W^l + b^l with Ahat = D~^-1/2 (A + I) D~^-1/2,
 *                D~ = local degree + 1 (Kipf & Welling's renormalised adjacency); one weight
 *                matrix W[d_l][d_{l+1}] per layer instead of Ws, Wn.
 *   norm = 1     hidden layers: U = gamma * (Z - mean) / sqrt(var + 1e-5) + beta over the row's
 *                features (biased variance), parameters gamma[d_{l+1}], beta[d_{l+1}].
 *   act = 1      hidden layers: H = U if U > 0 else a * U, one learnable slope a per layer.
 * The last layer has neither.  Parameter order inside a layer: weight matrices, b, then
 * (hidden layers only) gamma, beta if norm = 1, then a if act = 1.                          */
typedef struct {
    int32_t L;
    int32_t dims[RTMA_MAX_LAYERS + 1];
    int32_t gemm_dtype; /* 0: fp32-accurate products; 1: bf16 operands, fp32 accumulate   */
    float lr;
    int32_t encoder;    /* 0: GraphSAGE-mean; 1: GCN                                        */
    int32_t act;        /* 0: ReLU; 1: PReLU                                                */
    int32_t norm;       /* 0: none; 1: Layer Normalization before the activation            */
} rtma_model_desc;

int64_t rtma_param_count(const rtma_model_desc* model);

/* Optional record of one step's intermediates, for verification.  Any pointer may be NULL.
 * acts: for part 0..M-1 in turn, for l = 0..L-1: Abar H^l [n_p x d_l] then H^{l+1}
 * [n_p x d_{l+1}] (post-ReLU; the logits for l = L-1), densely packed.  grads: [M][P], the
 * gradient that step applied.  step: which local step (0-based) to record.                */
typedef struct {
    float* acts;
    float* grads;
    int32_t step;
} rtma_taps;

/* Runs K local SGD steps on each of the M parts: W_i <- W_i - lr * grad L_i(W_i).
 *   part_offsets_host, edge_offsets_host  HOST arrays [M+1] (copies of the device outputs).
 *   rowptr_out, col_out                   as produced by rtma_build_induced_csr.  The
 *                                         subgraphs must be symmetric (undirected graph,
 *                                         both directions stored), as the paper's "simple
 *                                         graph" is; symmetric != 1 is RTMA_ERR_UNSUPPORTED.
 *                                         The claim is verified on the device (a hash sum over
 *                                         the entries against one over the reversed entries):
 *                                         if it does not hold, the next rtma_check returns
 *                                         RTMA_ERR_INVALID_ARG and the parameters written by
 *                                         the call are not to be used.
 *   Xp [n][dims[0]] float, yp [n] int32   features / labels in partition order.
 *   params [M][P]                         in/out, one replica per trainer.
 *   loss_out [M][K] float or NULL         loss of every step of every trainer.
 *   streams  HOST array of M cudaStream_t: trainer i runs on streams[i].  Trainers that
 *            share a stream are batched into common launches; distinct streams run
 *            concurrently.  The call returns once everything is enqueued; while it sets
 *            up it waits for each stream once or twice unless rtma_set_dense_aggregation(ctx, 0).
 * Scratch is taken from the context (grows if needed).  A part may hold at most 2^31 - 1
 * nodes (RTMA_ERR_INVALID_ARG) and 2^31 - 1 kept entries (RTMA_ERR_OVERFLOW).               */
int32_t rtma_local_steps(rtma_ctx* ctx, const rtma_model_desc* model, int32_t M,
                         const int64_t* part_offsets_host, const int64_t* edge_offsets_host,
                         const int64_t* rowptr_out, const int32_t* col_out, int32_t symmetric,
                         const float* Xp, const int32_t* yp, float* params, int32_t K,
                         float* loss_out, const rtma_taps* taps, void* const* streams);

/* rtma_local_steps on features that are still in the graph's node order: X [n][dims[0]] as the
 * caller holds it, perm [n] from rtma_partition; row i of the partition order is X[perm[i]] ("load
 * G_train^(i)", Algorithm 2, done while the features are brought into the layout of the products).
 * Saves the rtma_gather_rows pass over the features and its copy in partition order.  yp stays in
 * partition order (rtma_gather_rows on the labels).  Everything else, and the result bit for bit,
 * as rtma_local_steps given rtma_gather_rows(X, perm).                                        */
int32_t rtma_local_steps_gathered(rtma_ctx* ctx, const rtma_model_desc* model, int32_t M,
                                  const int64_t* part_offsets_host, const int64_t* edge_offsets_host,
                                  const int64_t* rowptr_out, const int32_t* col_out, int32_t symmetric,
                                  const float* X, const int32_t* perm, const int32_t* yp, float* params,
                                  int32_t K, float* loss_out, const rtma_taps* taps, void* const* streams);

/* Local training with a step count of its own for every trainer.  Aggregation is triggered by
 * wall time, not by a step count (Sec. 3.1), so trainers arrive at an aggregation with
 * different numbers of finished steps (Sec. 3.1 and Table 3 report up to 28.8% fewer on the slowest one):
 * trainer i runs steps_host[i] steps.  steps_host[i] = 0 is a trainer that did not run at all,
 * e.g. one that failed to start (Sec. 4.5): its replica is left untouched and it takes neither
 * scratch nor launches.
 *   steps_host  HOST array [M], every entry >= 0.
 *   loss_out    [M][loss_stride] float or NULL, loss_stride >= max_i steps_host[i]; entries
 *               [i][s] with s >= steps_host[i] are not written.
 * Everything else as for rtma_local_steps, which is this call with every entry equal to K and
 * loss_stride = K.  Trainers that have finished drop out of the later launches.              */
int32_t rtma_local_steps_var(rtma_ctx* ctx, const rtma_model_desc* model, int32_t M,
                             const int64_t* part_offsets_host, const int64_t* edge_offsets_host,
                             const int64_t* rowptr_out, const int32_t* col_out, int32_t symmetric,
                             const float* Xp, const int32_t* yp, float* params,
                             const int32_t* steps_host, int32_t loss_stride, float* loss_out,
                             const rtma_taps* taps, void* const* streams);

/* ---- link prediction (Sec. 4.1 "Link Prediction Decoder", "Mini-batch and Negative Sampling";
 * App. "Formulation of MLP Decoder") ---------------------------------------------------------
 * The paper's own task.  The encoder is `model` (any variant); its last layer outputs the node
 * embeddings r [dims[L]] instead of class scores.  For a pair (u, v): e^0 = r_u (.) r_v
 * (element-wise), e^{k+1} = PReLU_k(e^k Theta^k) for the hidden decoder layers, the last layer
 * gives the scalar score s = e^{Kd-1} Theta^{Kd-1} (no biases, as in the paper's formula); the
 * link probability is sigmoid(s) and the loss the binary cross-entropy averaged over the part's
 * pairs (label 1: an edge of the training subgraph, 0: a sampled pair (u, v')).  Pairs and labels
 * are INPUTS (the paper draws them at random; drawing is the caller's business), as local ids of
 * the part.  The encoder runs on the whole part (no neighbour sampling).
 *   decoder     Kd layers, ddims[0] = dims[L], ddims[Kd] = 1.
 *   parameters  [M][P], P = rtma_link_param_count(): the encoder's parameters, then Theta^0
 *               [ddims[0]][ddims[1]], slope_0, Theta^1, slope_1, ..., Theta^{Kd-1} (no slope).
 *   pair_offsets_host  HOST [M+1]: part p's pairs are pair_u/pair_v/pair_label[pair_offsets[p] ..).
 *   loss_out [M][K] or NULL.  record_step >= 0: at that step grads_out [M][P] (or NULL) receives
 *   the gradient applied, emb_out [n][dims[L]] (or NULL) the embeddings, score_out [pairs] (or
 *   NULL) the scores.  Everything else as for rtma_local_steps; all trainers run K steps on the
 *   same pairs (a caller that wants a fresh mini-batch per step calls with K = 1).
 * The gradient of the embeddings is accumulated with floating-point atomics: its last bits, and
 * with them the result, can differ between runs (unlike rtma_local_steps).                   */
typedef struct {
    int32_t Kd;
    int32_t ddims[RTMA_MAX_LAYERS + 1];
} rtma_decoder_desc;

int64_t rtma_link_param_count(const rtma_model_desc* model, const rtma_decoder_desc* decoder);

int32_t rtma_link_steps(rtma_ctx* ctx, const rtma_model_desc* model, const rtma_decoder_desc* decoder,
                        int32_t M, const int64_t* part_offsets_host, const int64_t* edge_offsets_host,
                        const int64_t* rowptr_out, const int32_t* col_out, int32_t symmetric,
                        const float* Xp, const int64_t* pair_offsets_host, const int32_t* pair_u,
                        const int32_t* pair_v, const int32_t* pair_label, float* params, int32_t K,
                        float* loss_out, int32_t record_step, float* grads_out, float* emb_out,
                        float* score_out, void* const* streams);

/* ---- neighbour sampling (Sec. 4.1 "Mini-batch and Negative Sampling") ---------------------
 * One hop of the GraphSAGE neighbour sampler that shrinks the message-flow graph of a mini-batch, on
 * one part's induced subgraph (rowptr = the part's n+1 zero-based offsets inside rowptr_out, col =
 * its columns inside col_out).  The paper names the sampler and gives neither fan-outs nor the draw;
 * both are inputs here.  Every frontier node with at most `fanout` entries keeps them all, otherwise
 * it keeps the `fanout` entries with the smallest keys
 *     key = S(S(seed ^ ((hop + 1) << 48)) ^ ((v << 32) | position)),   S = one SplitMix64 step
 * (equal keys: the smaller position first): a uniform sample without replacement that depends only
 * on (seed, hop, node, position).  Start with the distinct end points of the batch's pairs as the
 * frontier and hop = 0; call again with next_frontier as the frontier and hop + 1, once per layer.
 *   frontier      [frontier_size] int32, ascending and distinct local ids.
 *   block_rowptr  [frontier_size + 1] int64: the hop's block, one row per frontier node.
 *   block_col     int32, room for sum_v min(deg(v), fanout) <= frontier_size * fanout entries:
 *                 positions in next_frontier, a row's entries in the order they have in the graph.
 *   next_frontier [n] int32 (room for every node): ascending union of the frontier and the kept
 *                 neighbours; next_size [1] int64 (device) receives its length.
 * Read next_size back (after draining the stream) before the next hop.  The result is unique: no
 * atomics on data, equal bit for bit from run to run.                                          */
int32_t rtma_sample_hop(rtma_ctx* ctx, int64_t n, const int64_t* rowptr, const int32_t* col,
                        int64_t frontier_size, const int32_t* frontier, int32_t fanout, uint64_t seed,
                        int32_t hop, int64_t* block_rowptr, int32_t* block_col, int32_t* next_frontier,
                        int64_t* next_size, void* stream);

/* ---- R2: aggregation (Algorithm 1, phi = plain average; Algorithm 2, overwrite) ---------
 * Wbar[j] = (1/M) sum_i params[i][j]; every replica is overwritten with Wbar; global_out
 * [P] (or NULL) also receives it.  M = 1 leaves the parameters unchanged.                 */
int32_t rtma_aggregate(rtma_ctx* ctx, float* params, int64_t P, int32_t M, float* global_out,
                       void* stream);

/* Aggregation when some trainers are offline (Sec. 4.5: training continues with the remaining
 * trainers): Wbar[j] = (1/|A|) sum_{i in A} params[i][j], A = { i : active_host[i] != 0 }.
 * Every replica, the inactive ones included, is overwritten with Wbar, as a trainer that
 * comes back would receive it.  active_host: HOST array [M] of bytes; an empty A is
 * RTMA_ERR_INVALID_ARG.  With every byte set this is rtma_aggregate, bit for bit.            */
int32_t rtma_aggregate_masked(rtma_ctx* ctx, float* params, int64_t P, int32_t M,
                              const uint8_t* active_host, float* global_out, void* stream);

/* The last local step fused with the aggregation: Wbar = (1/M) sum_i (params[i] - lr *
 * grads[i]), written to every replica (and global_out).  grads [M][P].                    */
int32_t rtma_sgd_aggregate(rtma_ctx* ctx, float* params, const float* grads, float lr, int64_t P,
                           int32_t M, float* global_out, void* stream);

/* ---- instrumentation --------------------------------------------------------------------
 * The library counts its kernel launches per class (RTMA_KERNEL_CLASSES classes, named by
 * rtma_kernel_class_name).  rtma_profile(ctx, 1) additionally brackets every launch with CUDA
 * events on the launching stream; rtma_profile_read synchronises the device, writes the time
 * summed per class (ms [RTMA_KERNEL_CLASSES], milliseconds; zeros if profiling was off) and the
 * launch counts (launches [RTMA_KERNEL_CLASSES]) since the previous read, and resets both.
 * Either output may be NULL.  The paper has no counterpart; these feed the roofline report.  */
#define RTMA_KERNEL_CLASSES 21
int32_t rtma_profile(rtma_ctx* ctx, int32_t enable);
int32_t rtma_profile_read(rtma_ctx* ctx, double* ms, int64_t* launches);
const char* rtma_kernel_class_name(int32_t cls);

/* Self-test of the device-side failure path.  Every wait inside the library's kernels is
 * bounded: a wait that runs out raises the context's device error word, the kernel winds down and
 * the next rtma_check returns RTMA_ERR_TIMEOUT, leaving the context usable.  This call launches a
 * one-block kernel whose wait can never be satisfied (a barrier nothing arrives at, about a
 * thousand polls) so that the path can be exercised without faulting or hanging the device.
 * The paper has no counterpart.                                                             */
int32_t rtma_selftest_wait_timeout(rtma_ctx* ctx, void* stream);

/* ---- the whole path on HOST buffers (Sec. 3: partition, Algorithm 2, Algorithm 1) --------
 * Every pointer here is a HOST pointer (pageable or pinned).  Copies the graph (CSR as for
 * rtma_build_induced_csr), group_id_h (NULL = RandomTMA), features X_h [n][dims[0]], labels
 * y_h [n] and the common initial parameters params0_h [P] to the device, runs rtma_partition
 * (rtma_partition_grouped when super-node ids are given), rtma_build_induced_csr, rtma_gather_rows (labels), then R rounds of (rtma_local_steps_gathered with K steps on
 * every part, rtma_aggregate), and copies back params_out_h [P] (the averaged parameters),
 * loss_out_h [R][M][K] (or NULL) and kept_cut_h [2] (or NULL).  The graph must be undirected
 * with both directions stored.  The device copies of the inputs live in buffers the context
 * keeps between calls (allocated with cudaMalloc when a call needs more than the last, freed by
 * rtma_destroy).  The graph is copied first; features, labels and parameters follow on a stream
 * of the context's own while the partition and subgraph kernels run.  SYNCHRONISES the stream
 * before returning.                                                                         */
int32_t rtma_train_host(rtma_ctx* ctx, int64_t n, int32_t rowptr_is_64, const void* rowptr_h,
                        const int32_t* col_h, const int32_t* group_id_h, const float* X_h,
                        const int32_t* y_h, const rtma_model_desc* model, int32_t M, uint64_t seed,
                        int32_t K, int32_t R, const float* params0_h, float* params_out_h,
                        float* loss_out_h, int64_t* kept_cut_h, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RTMA_H_ */
