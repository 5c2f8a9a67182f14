/*
 * embedpart.h -- C ABI of the B200 (sm_100a) library for the data-parallel hot path of
 * embedding-driven graph partitioning:
 *
 *   ep_kmeans             Lloyd K-Means over dense node embeddings -> partition of every vertex
 *                         (Algorithm 3, the clustering step P <- KMeans(E, k))
 *   ep_partition_quality  edge cut and per-partition loads of a partition over a CSR graph
 *                         (Section 2.1.1, Eq. 1 "edge-cut ratio" and Eq. 2 "vertex balance")
 *   ep_reorder            partition-ordered vertex relabelling for graph reordering
 *                         (Section 4.5.1: vertices of the same partition get consecutive ids)
 *
 * Conventions shared by every call
 *   - Pointers marked [dev] are CUDA device pointers on the context's device, owned by the
 *     caller; the library neither frees nor keeps them after the call.  Pointers marked [host]
 *     are ordinary host pointers.  Inputs are never modified.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL = default stream)
 *     and the call returns without waiting.  Outputs are valid once the stream has drained.
 *   - `workspace` [dev] is scratch the caller provides; its minimum size comes from the matching
 *     *_workspace_bytes query, it must be 256-byte aligned, and its contents are undefined on
 *     entry and exit.  Two calls that overlap on the GPU must not share a workspace.
 *   - The return value is a status code (EP_OK = 0).  Argument errors are found on the host before
 *     anything is launched.  Errors only the device can see (an out-of-range label or column
 *     index, a non-monotone row pointer, a bounded device wait that ran out) never fault: the
 *     offending element is skipped, a device status word is raised, and ep_poll_status returns
 *     it after the caller has synchronised.
 *   - No function prints, aborts or throws.  Nothing falls back to the CPU: on a device that is
 *     not compute capability 10.x, ep_create fails with EP_ERR_UNSUPPORTED.
 */
#ifndef EMBEDPART_H
#define EMBEDPART_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    EP_OK = 0,
    EP_ERR_INVALID_ARG = 1, /* null or misaligned pointer, size out of range */
    EP_ERR_UNSUPPORTED = 2, /* device is not sm_100, or a shape the library does not handle */
    EP_ERR_WORKSPACE = 3,   /* workspace too small or misaligned */
    EP_ERR_BAD_INDEX = 4,   /* device saw a label outside [0,K), a column outside [0,N) or a bad row pointer */
    EP_ERR_TIMEOUT = 5,     /* a bounded device-side wait expired */
    EP_ERR_CUDA = 6         /* a CUDA runtime or driver call failed; see ep_last_error */
};

/* Integer knobs for ep_set_option. */
enum {
    EP_OPT_KMEANS_PATH = 1, /* 0 = choose by shape (default), 1 = CUDA-core kernels only, 2 = tensor-core
                               (tcgen05) kernels wherever the shape allows */
    EP_OPT_PROFILE = 2,     /* 1 = bracket the main kernels with CUDA events on the launching stream
                               (read with ep_profile_read); 0 = off (default) */
    EP_OPT_TIMER_GROUP = 3, /* 0..3: calls made while group g is selected log into timers
                               g * EP_TIMER_COUNT + timer, so a caller can tell two calls apart */
    EP_OPT_KMEANS_CAND_MB = 4, /* 1..32768 (default 1024): upper bound in MiB of the candidate-key buffer the
                               tensor-core path keeps in the workspace (64 bytes per row and 1024 centroids);
                               rows are processed in chunks that fit it (never less than one pass of the
                               grid), and fewer, longer chunks run faster.  Set it before the workspace
                               query: it changes the answer */
    EP_OPT_QUALITY_SLICE_KB = 5 /* 1..4194304 (default 57344 = 56 MiB): ep_partition_quality gathers the label of
                               every entry's target; when the repacked labels of all vertices take more than this,
                               the vertex range is cut into up to 8 slices of at most this size and the column ids
                               are streamed once per slice, so that a slice's labels stay in the L2.  The result
                               does not depend on it */
    ,
    EP_OPT_KMEANS_ITERATIONS_PER_LAUNCH = 6 /* the fused small-K tensor-core pass (2 <= K <= 64): 0 (default) or 2 = all
                               Lloyd iterations of a call inside one launch, the blocks updating the centroids themselves
                               between grid-wide barriers; 1 = one launch per iteration plus the update kernel.  The
                               labels do not depend on it; centroids may differ in the last bit (another fixed order of
                               the fp64 fold) */
};

/* Timers kept while EP_OPT_PROFILE is 1. */
enum {
    EP_TIMER_KMEANS_ASSIGN = 0,  /* the assign(-and-accumulate) kernel of every Lloyd iteration; on the
                                    tensor-core path the screening kernel (one interval per row chunk) */
    EP_TIMER_KMEANS_UPDATE = 1,  /* everything else of an iteration: grouping, sums, centroid update */
    EP_TIMER_EDGE_CUT = 2,       /* the tiled edge-cut kernel */
    EP_TIMER_QUALITY_PREP = 3,   /* label repacking, partition loads, tile start rows */
    EP_TIMER_REORDER = 4,        /* all kernels of ep_reorder */
    EP_TIMER_KMEANS_RESOLVE = 5, /* tensor-core path: the fp32 kernel that decides the labels */
    EP_TIMER_GRAPH_BANDWIDTH = 6, /* all kernels of ep_graph_bandwidth */
    EP_TIMER_RELABEL = 7,        /* all kernels of ep_relabel_graph and ep_permute_rows */
    EP_TIMER_BALANCE = 8,        /* the kernels of ep_migrate / ep_balance other than the sort */
    EP_TIMER_COUNT = 9
};

typedef struct ep_ctx ep_ctx; /* opaque: device id, device properties, device status word, options */

/* Creates a context bound to CUDA device `device`.  Allocates a few bytes of device memory for the
 * status word.  Fails with EP_ERR_UNSUPPORTED unless the device is compute capability 10.x. */
int ep_create(ep_ctx **out, int device);
/* Releases the context.  The caller must have drained every stream that used it. */
int ep_destroy(ep_ctx *ctx);
/* Static, human-readable name of a status code. */
const char *ep_status_string(int status);
/* Text of the most recent host-side failure on this context ("" if none). */
const char *ep_last_error(const ep_ctx *ctx);
/* Reads and clears the device status word.  Synchronises the device; returns EP_OK or the most
 * severe EP_ERR_* raised by kernels since the last poll. */
int ep_poll_status(ep_ctx *ctx);
int ep_set_option(ep_ctx *ctx, int option, int value);
int ep_get_option(const ep_ctx *ctx, int option, int *value /* [host] */);
/* Sum of the event-timed durations (milliseconds) and the number of timed intervals recorded for
 * `timer` (group * EP_TIMER_COUNT + one of the EP_TIMER_* ids) since it was last read; waits for
 * the recorded events, then clears the timer.  total_ms and intervals are [host] and may be NULL. */
int ep_profile_read(ep_ctx *ctx, int timer, double *total_ms, int64_t *intervals);
/* Number of kernels this context has launched since it was created. */
int64_t ep_launch_count(const ep_ctx *ctx);
/* Diagnostic counters kept while EP_OPT_PROFILE is 1; synchronises the device, copies the 8 counters to
 * out [host, 8 x int64] and clears them.  Tensor-core K-Means paths: [0] rows screened, [1] centroids the
 * large-K path re-evaluated singly in fp32, [2] groups of 128 centroids it re-evaluated whole, [3] rows the
 * fused small-K kernel left undecided by its screening, [4] rows the large-K screening kernel left to the fp32
 * kernel, [5] and [6] (one launch for all iterations only) clocks block 0 spent assigning and accumulating /
 * meeting the other blocks and updating centroids; [7] is reserved. */
int ep_debug_counters(ep_ctx *ctx, int64_t *out);

/* Self-test of the bounded device wait (no counterpart in the paper: a property of this library).  Every wait
 * inside the tensor-core kernels gives up after a number of clocks and makes its kernel report EP_ERR_TIMEOUT
 * instead of hanging.  This call launches one small block whose first warp waits, for at most limit_clocks, on a
 * barrier that nothing ever completes, and whose second warp waits on the same barrier with the library's ordinary
 * limit (about 2 s) and has to leave when the first gives up.  Afterwards ep_poll_status returns EP_ERR_TIMEOUT
 * (once), and waited [dev, 3 x int64] holds the clocks either warp waited and, in [2], a bit per warp whose wait
 * claimed success (0 expected).  limit_clocks in [1e3, 2e8].  Nothing faults or spins without end. */
int ep_selftest_wait_timeout(ep_ctx *ctx, int64_t limit_clocks, int64_t *waited, void *cuda_stream);

/* Yardstick for the label gather of ep_partition_quality (Section 2.1.1, Eq. 1 needs the label of every entry's
 * target; the paper has no counterpart to this call).  Streams colidx exactly as the edge-cut pass does, gathers one
 * byte table[colidx[e]] per entry and sums the bytes: the edge-cut pass without its own work, i.e. the rate at which
 * this GPU serves such gathers.  cluster_size = 0: the table is read from global memory (L1 / L2), as the pass reads
 * labels that do not fit in shared memory; cluster_size = -1: the same table read through a texture object, i.e. by
 * the texture units instead of the load/store unit (the table must then be aligned as textures are, 512 bytes, and
 * no longer than the widest linear texture, else EP_ERR_INVALID_ARG / EP_ERR_UNSUPPORTED; the context keeps the
 * texture object of the last table until another table comes or the context is destroyed); cluster_size = 2, 4, 8
 * or 16: the table is first spread over the shared memory of thread-block clusters of that size and every lookup is
 * a ld.shared::cluster from the block that holds the vertex's slice (EP_ERR_UNSUPPORTED when N bytes do not fit
 * cluster_size blocks, or no such cluster fits the device).
 *   colidx [dev] nnz int32, 16-byte aligned; entries outside [0, N) are skipped
 *   table  [dev] N bytes;  sum [dev] out, 1 uint64: sum of the gathered bytes.  Asynchronous; time it with events. */
int ep_probe_gather(ep_ctx *ctx, const int32_t *colidx, int64_t nnz, const uint8_t *table, int64_t N,
                    int32_t cluster_size, uint64_t *sum, void *cuda_stream);

/* --------------------------------------------------------------------------------------------
 * ep_kmeans -- Lloyd K-Means (Algorithm 3, the clustering step).
 *
 * Squared Euclidean distance; exactly `iters` iterations from the given initial centroids, no
 * early stop.  In iteration t every row is assigned to its nearest centroid of C_{t-1} (of several
 * equidistant centroids the lowest index wins), then every centroid becomes the mean of its rows;
 * a centroid that received no row keeps its previous value.  Returned are the assignment of the
 * last iteration (made against C_{iters-1}) and C_iters, so each non-empty centroid is the mean of
 * the rows carrying its label.  iters == 0 assigns the rows against init_centroids and returns
 * those centroids unchanged.
 *
 *   emb            [dev] N x d fp32, row-major, 16-byte aligned
 *   N              rows, 1 <= N < 2^31
 *   d              columns, a multiple of 4 in [4, 1024]
 *   K              clusters, 1 <= K <= min(N, 65536)
 *   iters          >= 0
 *   init_centroids [dev] K x d fp32 row-major
 *   assign         [dev] out, N int32 in [0, K)
 *   centroids      [dev] out, K x d fp32 row-major (may alias init_centroids)
 *   objective      [dev] out or NULL: max(iters,1) doubles; entry t-1 is
 *                  J_t = sum_i |x_i - C_{t-1}[a_i]|^2 of iteration t
 *
 * Distances are evaluated as |c|^2 - 2 x.c in fp32 (on the tensor-core path a TF32 product screens
 * the candidates and every row whose two best scores are closer than the TF32 error bound is
 * re-evaluated in fp32).  Sums for the means are fp32 per thread block and fp64 across blocks, in a
 * fixed order: the result is the same from run to run on the same device.  A row holding NaN gets
 * some valid label and poisons that centroid; nothing faults.
 */
size_t ep_kmeans_workspace_bytes(const ep_ctx *ctx, int64_t N, int32_t d, int32_t K); /* 0 = invalid shape */
int ep_kmeans(ep_ctx *ctx, const float *emb, int64_t N, int32_t d, int32_t K, int32_t iters,
              const float *init_centroids, int32_t *assign, float *centroids, double *objective,
              void *workspace, size_t workspace_bytes, void *cuda_stream);

/* --------------------------------------------------------------------------------------------
 * ep_kmeans_sampled -- sampling-based clustering (Section 5, "Implementation": the centroids are
 * computed from a sample of the embeddings, 2^9 per cluster in the paper; every embedding is
 * then assigned to its nearest centroid).
 *
 * Three steps on the stream: the rows sample_rows of emb are gathered into the workspace;
 * `iters` >= 1 Lloyd iterations run over them from init_centroids (exactly as ep_kmeans);
 * one assign-only pass labels all N rows against the resulting centroids.  Unlike ep_kmeans,
 * the labels returned are those of the final centroids.
 *
 *   emb, N, d, K, init_centroids, centroids: as for ep_kmeans
 *   sample_rows [dev] M int64 row numbers in [0, N), distinct (not checked);  K <= M <= N
 *   assign      [dev] out, N int32
 * A row number outside [0, N) raises EP_ERR_BAD_INDEX in the device status word and is read as
 * row 0.  ep_gather_rows is the first step on its own: out[i] = emb[rows[i]].
 */
size_t ep_kmeans_sampled_workspace_bytes(const ep_ctx *ctx, int64_t N, int32_t d, int32_t K, int64_t M);
int ep_kmeans_sampled(ep_ctx *ctx, const float *emb, int64_t N, int32_t d, int32_t K, int32_t iters,
                      const int64_t *sample_rows, int64_t M, const float *init_centroids, int32_t *assign,
                      float *centroids, void *workspace, size_t workspace_bytes, void *cuda_stream);
int ep_gather_rows(ep_ctx *ctx, const float *emb, int64_t N, int32_t d, const int64_t *rows, int64_t M,
                   float *out /* [dev] M x d, 16-byte aligned */, void *cuda_stream);

/* --------------------------------------------------------------------------------------------
 * ep_partition_quality -- edge cut and partition loads (Eq. 1 numerator, Eq. 2 operands).
 *
 *   edge_cut         = number of stored CSR entries (u -> v) with assign[u] != assign[v]; entries
 *                      count as stored (both directions of a symmetric graph, duplicates each
 *                      time, self-loops never)
 *   part_vertices[p] = number of vertices with assign[v] == p
 *   part_edges[p]    = sum of the out-degrees of those vertices
 * The caller forms ECR = edge_cut / nnz and balance = max(part_vertices) / (N / K).
 *
 *   rowptr   [dev] N+1 row offsets, int32 or int64 as rowptr_is_int64 says, rowptr[0] = 0,
 *            non-decreasing, rowptr[N] = nnz
 *   colidx   [dev] nnz int32 column ids in [0, N), 16-byte aligned
 *   assign   [dev] N int32 labels in [0, K)
 *   N, nnz   1 <= N < 2^31, 0 <= nnz < 2^62;  1 <= K <= 2^24
 *   edge_cut [dev] out, 1 uint64;  part_vertices, part_edges [dev] out, K int64 each
 * All arithmetic is integer, so the result does not depend on scheduling.
 */
size_t ep_quality_workspace_bytes(const ep_ctx *ctx, int64_t N, int64_t nnz, int32_t K);
int ep_partition_quality(ep_ctx *ctx, const void *rowptr, int32_t rowptr_is_int64, const int32_t *colidx,
                         int64_t nnz, const int32_t *assign, int64_t N, int32_t K, uint64_t *edge_cut,
                         int64_t *part_vertices, int64_t *part_edges, void *workspace,
                         size_t workspace_bytes, void *cuda_stream);

/* --------------------------------------------------------------------------------------------
 * ep_reorder -- partition-ordered relabelling (Section 4.5.1).
 *
 * perm lists the vertex ids sorted by (assign[v], v): partitions in ascending order, original
 * order inside a partition (a stable counting sort), so exactly one output is correct.
 *
 *   assign   [dev] N int32 labels in [0, K);  1 <= N < 2^31;  1 <= K <= 2^24
 *   perm     [dev] out, N int32: perm[new_id] = old vertex id
 *   inv_perm [dev] out or NULL, N int32: inv_perm[v] = new id of v (the paper's bijection pi)
 */
size_t ep_reorder_workspace_bytes(const ep_ctx *ctx, int64_t N, int32_t K);
int ep_reorder(ep_ctx *ctx, const int32_t *assign, int64_t N, int32_t K, int32_t *perm, int32_t *inv_perm,
               void *workspace, size_t workspace_bytes, void *cuda_stream);

/* --------------------------------------------------------------------------------------------
 * ep_graph_bandwidth -- average graph bandwidth of a vertex numbering (Section 4.5.1, Eq. 3-5).
 *
 * pi[v] is the new id of vertex v (the inv_perm of ep_reorder).  For every stored entry (v -> u)
 * the gap is |pi[v] - pi[u]| (Eq. 3); the vertex bandwidth beta_v is the largest gap over the
 * entries of row v (Eq. 4), 0 for a row without entries; the average graph bandwidth is
 * bandwidth_sum / N (Eq. 5), the division left to the caller so that the result stays an exact
 * integer.
 *
 *   rowptr   [dev] N+1 row offsets, int32 or int64 as rowptr_is_int64 says, rowptr[0] = 0,
 *            non-decreasing, rowptr[N] = nnz
 *   colidx   [dev] nnz int32 column ids in [0, N), 16-byte aligned
 *   pi       [dev] N int32 new ids in [0, 2^31); normally a bijection of [0, N), not checked
 *   N, nnz   1 <= N < 2^31, 0 <= nnz < 2^62
 *   bandwidth_sum    [dev] out, 1 uint64: sum of beta_v
 *   vertex_bandwidth [dev] out or NULL, N int32: beta_v
 * A column id outside [0, N) or a row pointer that steps backwards raises EP_ERR_BAD_INDEX in the
 * device status word; the entry is skipped.  Integer maxima and sums only, so the result does not
 * depend on scheduling.  The _host variant takes host pointers and an arena like the others.
 */
size_t ep_graph_bandwidth_workspace_bytes(const ep_ctx *ctx, int64_t N, int64_t nnz);
int ep_graph_bandwidth(ep_ctx *ctx, const void *rowptr, int32_t rowptr_is_int64, const int32_t *colidx,
                       int64_t nnz, const int32_t *pi, int64_t N, uint64_t *bandwidth_sum,
                       int32_t *vertex_bandwidth, void *workspace, size_t workspace_bytes, void *cuda_stream);
size_t ep_graph_bandwidth_host_arena_bytes(const ep_ctx *ctx, int64_t N, int64_t nnz, int32_t rowptr_is_int64);
int ep_graph_bandwidth_host(ep_ctx *ctx, const void *rowptr, int32_t rowptr_is_int64, const int32_t *colidx,
                            int64_t nnz, const int32_t *pi, int64_t N, uint64_t *bandwidth_sum,
                            int32_t *vertex_bandwidth, void *arena, size_t arena_bytes, void *cuda_stream);

/* --------------------------------------------------------------------------------------------
 * ep_relabel_graph, ep_permute_rows -- the graph and the embedding (or feature) rows stored under
 * the new numbering (Section 4.5.1: vertex ids are positions in memory; reordering relabels them).
 *
 * perm and inv_perm are the outputs of ep_reorder.  Row i of the new graph is row perm[i] of the
 * old one with every column id u replaced by inv_perm[u]; the entries of a row keep their stored
 * order, so exactly one output is correct.  ep_permute_rows writes out[i] = emb[perm[i]].
 *
 *   rowptr, colidx, nnz, N: as for ep_partition_quality
 *   perm, inv_perm [dev] N int32 each, inverse permutations of [0, N) (not checked beyond range)
 *   new_rowptr     [dev] out, N+1 offsets of the same width as rowptr
 *   new_colidx     [dev] out, nnz int32
 *   emb, out       [dev] N x d fp32 row-major, 16-byte aligned, d a multiple of 4 in [4, 1024]; not the same buffer
 * A value of perm or colidx outside [0, N) raises EP_ERR_BAD_INDEX in the device status word (the row
 * comes out empty, the id as 0).
 */
size_t ep_relabel_graph_workspace_bytes(const ep_ctx *ctx, int64_t N, int64_t nnz);
int ep_relabel_graph(ep_ctx *ctx, const void *rowptr, int32_t rowptr_is_int64, const int32_t *colidx, int64_t nnz,
                     const int32_t *perm, const int32_t *inv_perm, int64_t N, void *new_rowptr,
                     int32_t *new_colidx, void *workspace, size_t workspace_bytes, void *cuda_stream);
int ep_permute_rows(ep_ctx *ctx, const float *emb, int64_t N, int32_t d, const int32_t *perm, float *out,
                    void *cuda_stream);

/* --------------------------------------------------------------------------------------------
 * ep_migrate, ep_balance -- the migration policy M(P, S, C) (Algorithm 4: random migration in
 * proportion to free capacity) and the balancing loop of Algorithm 3 that applies it to one
 * vertex set until no partition holds more than C vertices of the set.  Algorithm 3 runs the
 * loop three times (training, validation and remaining vertices): three calls with three masks.
 *
 * One application: loads L_i = |{v in S : assign[v] = i}|; from every partition with L_i > C
 * the L_i - C vertices of S with the smallest degree leave (the degree is the row length; equal
 * degrees: the lower vertex id first); each goes to a partition with L_j < C, drawn with
 * probability (C - L_j) / F, F the total free capacity: vertex v goes to the partition whose
 * stretch holds t = floor(rand_words[v] * F / 2^32) when the free capacities are laid end to end
 * in ascending partition order.  Loads and probabilities are those from before the first move.
 * Random words are an input; the library draws no numbers.
 *
 *   rowptr      [dev] N+1 row offsets (int32 or int64), only the row lengths are used
 *   N, K        1 <= N < 2^31;  1 <= K <= 1024
 *   member      [dev] N bytes, non-zero = the vertex belongs to S; NULL = every vertex does
 *   capacity    C >= 0, the same for every partition (Algorithm 3 passes floor(beta |S| / K))
 *   max_degree  an upper bound of the row lengths; K * (max_degree + 1) must stay below 2^30
 *               (EP_ERR_UNSUPPORTED otherwise); a longer row raises EP_ERR_BAD_INDEX and its vertex stays
 *   rand_words  [dev] N uint32 (ep_migrate), max_rounds x N uint32, one row per round (ep_balance)
 *   assign      [dev] in/out, N int32 labels in [0, K)
 *   state       [dev] out or NULL, 4 int64: [0] vertices above capacity before the call, [1] F,
 *               [2] vertices moved, or -1 when there is no free capacity to move them to, [3] 0
 * ep_migrate is asynchronous like the other calls.  ep_balance synchronises the stream after every
 * round (it has to know whether another one is needed), stops as soon as no partition is above C,
 * writes the number of applications to *rounds_used [host] and returns EP_ERR_INVALID_ARG when C * K is
 * too small to hold S, EP_ERR_UNSUPPORTED when max_rounds applications were not enough.
 */
size_t ep_balance_workspace_bytes(const ep_ctx *ctx, int64_t N, int32_t K, int64_t max_degree);
int ep_migrate(ep_ctx *ctx, const void *rowptr, int32_t rowptr_is_int64, int64_t N, int32_t K, const uint8_t *member,
               int64_t capacity, int64_t max_degree, const uint32_t *rand_words, int32_t *assign, int64_t *state,
               void *workspace, size_t workspace_bytes, void *cuda_stream);
int ep_balance(ep_ctx *ctx, const void *rowptr, int32_t rowptr_is_int64, int64_t N, int32_t K, const uint8_t *member,
               int64_t capacity, int64_t max_degree, const uint32_t *rand_words, int32_t max_rounds, int32_t *assign,
               int32_t *rounds_used, void *workspace, size_t workspace_bytes, void *cuda_stream);

/* --------------------------------------------------------------------------------------------
 * ep_cluster_and_balance -- Phase 2 as a whole (Algorithm 3): P <- KMeans(E, k), then the balancing
 * loop for the training vertices, for the validation vertices and for the remaining ones, in that
 * order, each with its own capacity.  The calls above, made by the library in sequence.
 *
 *   emb, N, d, K, iters, init_centroids, assign, centroids: as for ep_kmeans
 *   rowptr, rowptr_is_int64, max_degree:                    as for ep_balance
 *   split       [dev] N bytes: 0 = training, 1 = validation, 2 = remaining vertex
 *   capacities  [host] 3 int64: C of each set (the paper uses floor(beta_x |V_x| / K))
 *   rand_words  [dev] 3 x max_rounds x N uint32: set s uses rows [s * max_rounds, (s + 1) * max_rounds)
 *   rounds_used [host] out or NULL, 3 int32
 * Synchronises the stream like ep_balance; errors as for ep_kmeans and ep_balance.
 */
size_t ep_cluster_and_balance_workspace_bytes(const ep_ctx *ctx, int64_t N, int32_t d, int32_t K, int64_t max_degree);
int ep_cluster_and_balance(ep_ctx *ctx, const float *emb, int64_t N, int32_t d, int32_t K, int32_t iters,
                           const float *init_centroids, const void *rowptr, int32_t rowptr_is_int64,
                           int64_t max_degree, const uint8_t *split, const int64_t *capacities,
                           const uint32_t *rand_words, int32_t max_rounds, int32_t *assign, float *centroids,
                           int32_t *rounds_used, void *workspace, size_t workspace_bytes, void *cuda_stream);

/* --------------------------------------------------------------------------------------------
 * Host-buffer variants.  Same operations and the same kernels; inputs and outputs are [host]
 * pointers.  Each call copies its inputs into `arena` (a [dev] scratch block of at least
 * *_host_arena_bytes bytes, 256-byte aligned, which also holds the kernel workspace), runs, and
 * copies the outputs back, all enqueued on `cuda_stream` with cudaMemcpyAsync: with page-locked
 * host buffers the call returns at once and the outputs are valid when the stream has drained;
 * with pageable buffers the copies block the calling thread as cudaMemcpyAsync documents.
 */
size_t ep_kmeans_host_arena_bytes(const ep_ctx *ctx, int64_t N, int32_t d, int32_t K, int32_t iters);
int ep_kmeans_host(ep_ctx *ctx, const float *emb, int64_t N, int32_t d, int32_t K, int32_t iters,
                   const float *init_centroids, int32_t *assign, float *centroids, double *objective,
                   void *arena, size_t arena_bytes, void *cuda_stream);
size_t ep_quality_host_arena_bytes(const ep_ctx *ctx, int64_t N, int64_t nnz, int32_t K, int32_t rowptr_is_int64);
int ep_partition_quality_host(ep_ctx *ctx, const void *rowptr, int32_t rowptr_is_int64, const int32_t *colidx,
                              int64_t nnz, const int32_t *assign, int64_t N, int32_t K, uint64_t *edge_cut,
                              int64_t *part_vertices, int64_t *part_edges, void *arena, size_t arena_bytes,
                              void *cuda_stream);
size_t ep_reorder_host_arena_bytes(const ep_ctx *ctx, int64_t N, int32_t K);
int ep_reorder_host(ep_ctx *ctx, const int32_t *assign, int64_t N, int32_t K, int32_t *perm, int32_t *inv_perm,
                    void *arena, size_t arena_bytes, void *cuda_stream);

/* --------------------------------------------------------------------------------------------
 * ep_partition_and_reorder_host -- the whole path on host buffers, every input uploaded once:
 * P <- KMeans(E, K) (Algorithm 3, the clustering step), its edge cut and loads (Section 2.1.1, Eq. 1 and 2), and the
 * partition-ordered numbering of Section 4.5.1, taken from a second clustering of the same embeddings with
 * reorder_K clusters (reordering wants many small clusters) or, with reorder_K = 0, from P itself.  The same
 * kernels as the separate calls, in this order on `cuda_stream`: uploads, ep_kmeans(K), ep_partition_quality,
 * ep_kmeans(reorder_K), ep_reorder, each result copied back as soon as it exists.  What it saves over four *_host
 * calls is the second upload of the embedding matrix and the upload of the labels.
 *
 *   emb, N, d, K, iters, init_centroids, assign, centroids:  as for ep_kmeans_host
 *   reorder_K, reorder_iters, reorder_init [host, reorder_K x d]: the second run; reorder_K = 0 = none
 *   rowptr, rowptr_is_int64, colidx, nnz, edge_cut, part_vertices, part_edges: as for ep_partition_quality_host
 *   reorder_assign [host] out or NULL, N int32: the labels of the second run
 *   perm, inv_perm [host] out (inv_perm may be NULL), N int32 each: as for ep_reorder_host
 *   arena [dev]: at least ep_partition_and_reorder_host_arena_bytes, 256-byte aligned
 */
size_t ep_partition_and_reorder_host_arena_bytes(const ep_ctx *ctx, int64_t N, int32_t d, int32_t K, int32_t reorder_K,
                                                 int64_t nnz, int32_t rowptr_is_int64);
int ep_partition_and_reorder_host(ep_ctx *ctx, const float *emb, int64_t N, int32_t d, int32_t K, int32_t iters,
                                  const float *init_centroids, int32_t reorder_K, int32_t reorder_iters,
                                  const float *reorder_init, const void *rowptr, int32_t rowptr_is_int64,
                                  const int32_t *colidx, int64_t nnz, int32_t *assign, float *centroids,
                                  uint64_t *edge_cut, int64_t *part_vertices, int64_t *part_edges,
                                  int32_t *reorder_assign, int32_t *perm, int32_t *inv_perm, void *arena,
                                  size_t arena_bytes, void *cuda_stream);

/* --------------------------------------------------------------------------------------------
 * ep_reorder_static -- ep_reorder without a workspace and without a context.  (The paper has no
 * counterpart to this call; it exists for the sake of callers, not of the method.)
 *
 * Some code that wants the permutation is not in a position to obtain device memory: a callback
 * running inside someone else's framework whose allocator it must not touch, a process whose
 * memory pool was sized and handed out at start-up, a latency-critical loop in which cudaMalloc's
 * implicit device synchronisation is unacceptable.  ep_reorder needs a workspace and ep_create
 * itself allocates a status word, so neither is usable there.  This variant performs the same
 * stable sort with the same kernel, but keeps its scratch (one row of digit counts per thread block
 * and the word the blocks meet on, about 1 MB) in an array compiled into the library.  Every GPU that
 * loads the library holds that array until the process ends, whether or not this function is ever called.
 *
 *   assign, perm, inv_perm   as for ep_reorder ([dev], caller-owned; inv_perm may be NULL)
 *   N                        1 <= N <= EP_REORDER_STATIC_MAX_N
 *   K                        1 <= K <= EP_REORDER_STATIC_MAX_K   (the one-pass range of the sort)
 *   device_status            [dev] out or NULL: one int32, set to EP_OK, or to EP_ERR_BAD_INDEX if a
 *                            label outside [0, K) was seen, or to EP_ERR_TIMEOUT if the blocks' bounded
 *                            wait for one another ran out (valid once the stream has drained).  With NULL
 *                            the word is kept inside the built-in array, where no call can read it: a
 *                            caller that wants to learn of bad labels must pass a word of its own
 *   cuda_stream              as elsewhere
 *
 * Works on the device that is current in the calling thread.  Returns EP_ERR_UNSUPPORTED when N or
 * K exceeds the limits above (nothing is launched), EP_ERR_INVALID_ARG for null or misaligned
 * pointers, EP_ERR_CUDA if a runtime call fails.  The function calls no cudaMalloc, cudaFree or
 * other allocating routine; it enqueues two 4-byte memsets and one kernel (a cooperative launch: its
 * blocks are resident together) on the stream.
 *
 * Every call looks up the device address of the built-in array; the first such look-up on a device
 * is a one-time set-up step of the CUDA runtime (it loads the library's code there): make that first
 * call outside of any stream capture.
 *
 * All calls on a device share the one array, and it keeps whatever the previous call left in it.
 * The function clears the two words that have to start at zero and its kernel overwrites every
 * count before reading it, so back-to-back calls on one stream are fine.  Two calls that can run on
 * the GPU at the same time (different streams, different host threads) would scribble over each
 * other's counts: order them yourself.
 */
#define EP_REORDER_STATIC_MAX_N 4194304 /* 2^22 vertices */
#define EP_REORDER_STATIC_MAX_K 256
int ep_reorder_static(const int32_t *assign, int64_t N, int32_t K, int32_t *perm, int32_t *inv_perm,
                      int32_t *device_status, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* EMBEDPART_H */
