/*
 * ep_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, fp64 CPU statement of what the EmbedPart hot path computes:
 *   - Lloyd K-Means over dense node embeddings  (Algorithm 3, the clustering step P <- KMeans(E, k))
 *   - edge cut and per-partition loads           (Section 2.1.1, Eq. 1 and Eq. 2)
 *   - the partition-ordered vertex permutation   (Section 4.5.1, "Adapting EmbedPart for Reordering")
 *   - the average graph bandwidth of a numbering (Section 4.5.1, Eq. 3, Eq. 4 and Eq. 5)
 *   - the graph and the embedding rows stored under the new numbering (Section 4.5.1)
 *   - the migration policy that balances the partitions (Algorithm 4, used by the balancing loops of Algorithm 3)
 *
 * Only tests, the smoke check and the CPU-baseline leg of the benchmark may call
 * this file.  It shares no code, header, table or helper with the CUDA library
 * and the CUDA library never calls it.
 *
 * Every function is pinned by CPU tests (brute force over all labelings, hand-
 * computed fixtures, closed forms, invariants, library special cases); none is
 * "parity unpinned".
 *
 * Arithmetic: every floating-point operation is IEEE double.  Embeddings and
 * initial centroids arrive as fp32 and are widened exactly.  Counters are 64-bit.
 * OpenMP, where used, only splits loops whose iterations are independent (or an
 * integer sum), so the result does not depend on the thread count.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/*
 * Assignment step of Lloyd's algorithm: every row goes to the centroid with the
 * smallest squared Euclidean distance, written in the direct form
 * sum_j (x_ij - c_kj)^2.  Centroids are scanned k = 0..K-1 with a strict '<',
 * so of several equidistant centroids the lowest index wins.
 *
 * best1[i] / best2[i] (either may be NULL) receive the smallest and the second
 * smallest distance of row i (best2 = +inf when K == 1); tests use them to find
 * rows whose two nearest centroids are too close to call in fp32.
 */
void oracle_assign(const float *emb, int64_t N, int32_t d,
                   const double *C, int32_t K,
                   int32_t *assign, double *best1, double *best2)
{
    int64_t i;
#pragma omp parallel for schedule(static)
    for (i = 0; i < N; ++i) {
        const float *x = emb + i * (int64_t)d;
        double m1 = INFINITY, m2 = INFINITY;
        int32_t a = 0;
        for (int32_t k = 0; k < K; ++k) {
            const double *c = C + (int64_t)k * d;
            double dist = 0.0;
            for (int32_t j = 0; j < d; ++j) {
                double diff = (double)x[j] - c[j];
                dist += diff * diff;
            }
            if (dist < m1) {
                m2 = m1;
                m1 = dist;
                a = k;
            } else if (dist < m2) {
                m2 = dist;
            }
        }
        assign[i] = a;
        if (best1) best1[i] = m1;
        if (best2) best2[i] = m2;
    }
}

/*
 * Lloyd K-Means, exactly `iters` iterations, no early stop (Algorithm 3, the clustering step
 * under the reading: squared Euclidean distance, explicit initial centroids,
 * full batch).
 *
 *   C_0 = init
 *   for t = 1..T:
 *       a_i  = argmin_k |x_i - C_{t-1}[k]|^2          (oracle_assign)
 *       J_t  = sum_i |x_i - C_{t-1}[a_i]|^2
 *       C_t[k] = mean of the rows with a_i = k, or C_{t-1}[k] when no row has a_i = k
 *
 * Returns the assignment of iteration T (made against C_{T-1}) together with
 * C_T, so every non-empty centroid is exactly the mean of the rows that carry
 * its label.  With iters == 0 the rows are assigned against C_0, centroids =
 * C_0 and objective[0] = the objective of that assignment.
 *
 * objective: max(iters,1) doubles, or NULL.  best1/best2: per-row two smallest
 * distances of the returned assignment, or NULL.
 * Returns 0, or -1 when scratch memory cannot be had.
 */
int oracle_kmeans(const float *emb, int64_t N, int32_t d, int32_t K, int32_t iters,
                  const float *init_centroids,
                  int32_t *assign, double *centroids, double *objective,
                  double *best1, double *best2)
{
    int64_t KD = (int64_t)K * d;
    double *prev = (double *)malloc(sizeof(double) * (size_t)KD);
    double *sum = (double *)malloc(sizeof(double) * (size_t)KD);
    int64_t *cnt = (int64_t *)malloc(sizeof(int64_t) * (size_t)K);
    double *m1 = best1 ? best1 : (double *)malloc(sizeof(double) * (size_t)N);
    if (!prev || !sum || !cnt || !m1) {
        free(prev); free(sum); free(cnt);
        if (!best1) free(m1);
        return -1;
    }
    for (int64_t q = 0; q < KD; ++q) centroids[q] = (double)init_centroids[q];

    int32_t T = iters > 0 ? iters : 1;
    for (int32_t t = 0; t < T; ++t) {
        memcpy(prev, centroids, sizeof(double) * (size_t)KD);
        oracle_assign(emb, N, d, prev, K, assign, m1, best2);

        double J = 0.0;
        for (int64_t i = 0; i < N; ++i) J += m1[i];
        if (objective) objective[t] = J;
        if (iters == 0) break;

        memset(sum, 0, sizeof(double) * (size_t)KD);
        memset(cnt, 0, sizeof(int64_t) * (size_t)K);
        for (int64_t i = 0; i < N; ++i) {
            int32_t a = assign[i];
            const float *x = emb + i * (int64_t)d;
            double *s = sum + (int64_t)a * d;
            for (int32_t j = 0; j < d; ++j) s[j] += (double)x[j];
            cnt[a] += 1;
        }
        for (int32_t k = 0; k < K; ++k) {
            if (cnt[k] > 0) {
                for (int32_t j = 0; j < d; ++j)
                    centroids[(int64_t)k * d + j] = sum[(int64_t)k * d + j] / (double)cnt[k];
            } /* an empty cluster keeps its previous centroid */
        }
    }
    free(prev); free(sum); free(cnt);
    if (!best1) free(m1);
    return 0;
}

/*
 * Edge cut and partition loads (Eq. 1 numerator; the operands of Eq. 2).
 *
 *   edge_cut         = number of stored CSR entries (u -> v) with pid(u) != pid(v)
 *   part_vertices[p] = |{v : pid(v) = p}|
 *   part_edges[p]    = sum of the out-degrees of the vertices in p
 *
 * Entries are counted as stored: a symmetric CSR counts an undirected cut edge
 * twice, a self-loop is never cut, a duplicate entry counts each time.
 */
void oracle_partition_quality(const int64_t *rowptr, const int32_t *colidx,
                              const int32_t *assign, int64_t N, int32_t K,
                              uint64_t *edge_cut, int64_t *part_vertices, int64_t *part_edges)
{
    int64_t cut = 0;
    int64_t u;
#pragma omp parallel for schedule(dynamic, 4096) reduction(+ : cut)
    for (u = 0; u < N; ++u) {
        int32_t pu = assign[u];
        for (int64_t e = rowptr[u]; e < rowptr[u + 1]; ++e)
            if (assign[colidx[e]] != pu) cut += 1;
    }
    *edge_cut = (uint64_t)cut;

    for (int32_t p = 0; p < K; ++p) { part_vertices[p] = 0; part_edges[p] = 0; }
    for (int64_t v = 0; v < N; ++v) {
        part_vertices[assign[v]] += 1;
        part_edges[assign[v]] += rowptr[v + 1] - rowptr[v];
    }
}

/*
 * Partition-ordered relabelling (Section 4.5.1): vertices of the same partition
 * get consecutive new ids.  Partitions come in ascending order and, inside a
 * partition, vertices keep their original order, i.e. perm lists the vertex ids
 * sorted by the pair (pid(v), v).  Written as a stable counting sort.
 *
 *   perm[new_id]   = old vertex id
 *   inv_perm[v]    = new id of vertex v        (the paper's pi; may be NULL)
 * Returns 0, or -1 when scratch memory cannot be had.
 */
int oracle_reorder(const int32_t *assign, int64_t N, int32_t K,
                   int32_t *perm, int32_t *inv_perm)
{
    int64_t *next = (int64_t *)calloc((size_t)K + 1, sizeof(int64_t));
    if (!next) return -1;
    for (int64_t v = 0; v < N; ++v) next[assign[v] + 1] += 1;
    for (int32_t p = 0; p < K; ++p) next[p + 1] += next[p];   /* next[p] = first new id of partition p */
    for (int64_t v = 0; v < N; ++v) {
        int64_t pos = next[assign[v]]++;
        perm[pos] = (int32_t)v;
        if (inv_perm) inv_perm[v] = (int32_t)pos;
    }
    free(next);
    return 0;
}

/*
 * Graph bandwidth of a vertex numbering (Section 4.5.1).  pi[v] is the new id of
 * vertex v, a bijection of [0, N).
 *
 *   gap of an entry (v -> u)      xi = |pi[v] - pi[u]|                       (Eq. 3)
 *   vertex bandwidth              beta_v = max of xi over the entries of row v (Eq. 4)
 *   average graph bandwidth       (1/N) sum over v of beta_v                   (Eq. 5)
 *
 * The neighbours n(v) are the stored entries of row v; a vertex without entries
 * has an empty maximum, read as 0 (it touches no other vertex); a self-loop has
 * gap 0.  The sum is returned as an exact integer, the caller divides by N;
 * vertex_bandwidth (may be NULL) receives beta_v.
 */
void oracle_graph_bandwidth(const int64_t *rowptr, const int32_t *colidx, const int32_t *pi,
                            int64_t N, uint64_t *bandwidth_sum, int32_t *vertex_bandwidth)
{
    int64_t total = 0;
    int64_t v;
#pragma omp parallel for schedule(dynamic, 4096) reduction(+ : total)
    for (v = 0; v < N; ++v) {
        int64_t beta = 0;
        for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) {
            int64_t xi = (int64_t)pi[v] - (int64_t)pi[colidx[e]];
            if (xi < 0) xi = -xi;
            if (xi > beta) beta = xi;
        }
        if (vertex_bandwidth) vertex_bandwidth[v] = (int32_t)beta;
        total += beta;
    }
    *bandwidth_sum = (uint64_t)total;
}

/*
 * The graph stored under a new numbering (Section 4.5.1: the ids of the vertices are their
 * positions in memory, and reordering relabels them).  perm[new_id] = old id and
 * inv_perm[old id] = new id, as oracle_reorder returns them.  Row i of the new graph is row
 * perm[i] of the old one with every column id u replaced by inv_perm[u]; the entries of a row keep
 * their stored order (the paper does not ask for sorted rows), so exactly one output is correct.
 */
void oracle_relabel_graph(const int64_t *rowptr, const int32_t *colidx, const int32_t *perm,
                          const int32_t *inv_perm, int64_t N, int64_t *new_rowptr, int32_t *new_colidx)
{
    new_rowptr[0] = 0;
    for (int64_t i = 0; i < N; ++i) {
        int64_t v = perm[i];
        int64_t at = new_rowptr[i];
        for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) new_colidx[at++] = inv_perm[colidx[e]];
        new_rowptr[i + 1] = at;
    }
}

/* Embedding (or feature) rows under the new numbering: out[i] = emb[perm[i]]. */
void oracle_permute_rows(const float *emb, int64_t N, int32_t d, const int32_t *perm, float *out)
{
    for (int64_t i = 0; i < N; ++i)
        memcpy(out + (size_t)i * d, emb + (size_t)perm[i] * d, sizeof(float) * (size_t)d);
}

/*
 * One application of the migration policy M(P, S, C) (Algorithm 4): random migration in
 * proportion to free capacity.
 *
 *   member[v] != 0   v belongs to the candidate set S (NULL: every vertex does)
 *   capacity         C, the same for every partition (Algorithm 3 passes beta |S| / k)
 *   rand_words[v]    the random number that vertex v uses if it is moved (uniform 32-bit words,
 *                    an input so that nothing here draws numbers)
 *
 * Steps, as the algorithm lists them: loads L_i = |{v in S : P(v) = i}|; overloaded O = {L_i > C},
 * underloaded U = {L_i < C}; free capacity f_i = C - L_i on U, F = their sum; from every i in O
 * the m_i = L_i - C vertices of S with the smallest degree are taken (equal degrees: the smaller
 * vertex id first; the degree is the row length); a taken vertex v goes to the partition of U
 * that the number t = floor(rand_words[v] * F / 2^32) falls into when the f_j of U are laid end to
 * end in ascending partition order, i.e. j is drawn with probability f_j / F.  Loads and
 * probabilities are those from before the first move.
 * Returns the number of vertices moved, -1 when there are overloaded partitions but no free
 * capacity, -2 when scratch memory cannot be had.
 */
typedef struct { int64_t deg; int64_t v; } oracle_deg_id;

static int oracle_deg_id_less(const void *a, const void *b)
{
    const oracle_deg_id *x = (const oracle_deg_id *)a, *y = (const oracle_deg_id *)b;
    if (x->deg != y->deg) return x->deg < y->deg ? -1 : 1;
    return x->v < y->v ? -1 : (x->v > y->v ? 1 : 0);
}

int64_t oracle_migrate(const int64_t *rowptr, int64_t N, int32_t K, const uint8_t *member, int64_t capacity,
                       const uint32_t *rand_words, int32_t *assign)
{
    int64_t *load = (int64_t *)calloc((size_t)K, sizeof(int64_t));
    int64_t *cum = (int64_t *)calloc((size_t)K, sizeof(int64_t));     /* free capacity of U up to and including j */
    oracle_deg_id *cand = (oracle_deg_id *)malloc(sizeof(oracle_deg_id) * (size_t)(N > 0 ? N : 1));
    if (!load || !cum || !cand) { free(load); free(cum); free(cand); return -2; }
    for (int64_t v = 0; v < N; ++v)
        if (!member || member[v]) load[assign[v]] += 1;
    int64_t F = 0, over = 0;
    for (int32_t j = 0; j < K; ++j) {
        if (load[j] < capacity) F += capacity - load[j];
        if (load[j] > capacity) over += load[j] - capacity;
        cum[j] = F;
    }
    int64_t moved = 0;
    if (over > 0 && F == 0) moved = -1;
    for (int32_t i = 0; i < K && moved >= 0; ++i) {
        if (load[i] <= capacity) continue;
        const int64_t m = load[i] - capacity;
        int64_t n = 0;
        for (int64_t v = 0; v < N; ++v)
            if ((!member || member[v]) && assign[v] == i) { cand[n].deg = rowptr[v + 1] - rowptr[v]; cand[n].v = v; ++n; }
        qsort(cand, (size_t)n, sizeof(oracle_deg_id), oracle_deg_id_less);
        for (int64_t s = 0; s < m; ++s) {
            const int64_t v = cand[s].v;
            const uint64_t t = ((uint64_t)rand_words[v] * (uint64_t)F) >> 32;
            int32_t j = 0;
            while ((uint64_t)cum[j] <= t) ++j;               /* first partition whose cumulative capacity exceeds t */
            assign[v] = j;
            ++moved;
        }
    }
    free(load); free(cum); free(cand);
    return moved;
}
