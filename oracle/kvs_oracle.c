/*
 * kvs_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, fp64 CPU statement of decode attention over a layer-shared
 * KV cache as KVSharer describes it.  It exists only so that tests, the smoke
 * check and the benchmark's CPU-baseline leg have something obviously correct
 * to compare the GPU library against.  It shares no code, header, table or
 * helper with the CUDA path and the CUDA path never calls it.
 *
 * What it follows, in the paper's own order:
 *   - Section 3 / Section 3.2 and the caption of Fig. 3: a sharing strategy Z
 *     is a fixed list saying which layers' KV caches are replaced by which
 *     other layers'; during the forward pass, when a layer's cache is to be
 *     replaced, the cache of the previously computed layer is copied to the
 *     current layer and the layer's remaining computation is unchanged.
 *   - Section 3.1 "Sharing Strategy Searching": the layer nearer the output is
 *     replaced by the layer nearer the input, so a source index is never
 *     larger than its target index.
 *   - Caption of the main-results table (Table 1): its Layer column is the
 *     number of layers that still compute a KV cache of their own, so a
 *     sharing layer computes (appends) nothing.
 *   - Section 1: the attention is the standard Transformer attention,
 *     softmax(q K^T / sqrt(d)) V, which the paper cites and does not restate.
 *
 * Readings where the paper is silent: no mask in decode (the one query is the
 * newest position and sees every cached row, its own included); a sharing
 * layer sees the current token of its source, because the source ran earlier
 * in the same forward pass; chains (a source that itself shares) are legal and
 * fall out of the literal copy in layer order; grouped-query heads map
 * q-head -> kv-head by integer division by the group size.
 *
 * Every cache here is a real, separate, per-layer array (L caches, never
 * L - #shared) and sharing is a literal deep copy, exactly as the text says.
 * That is deliberate: the GPU library replaces the copy by an indirection
 * table, and this file is the independent check of that replacement.
 *
 * Pinned by tests/test_oracle_pins.py (library SDPA in fp64 under the identity
 * map, brute force, closed forms, invariants, the paper's layer counts).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int L, Hq, Hkv, D, B;
    double scale;    /* 1/sqrt(D) unless the caller fixed another one        */
    int *share_map;  /* share_map[l] = layer whose cache layer l uses        */
    int **ulen;      /* ulen[l][b*Hkv+h]: cached tokens of that (sequence, head) of layer l;
                        equal across a layer until an intra-layer method evicts rows */
    int *cap;        /* allocated tokens per unit of layer l                 */
    double ***K;     /* K[l][b*Hkv+h] -> [cap][D] row-major                  */
    double ***V;
} oracle_state;

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---- single (sequence, q-head) attention: the definition itself ---------
 * out[d] = sum_j softmax_j(scale * q.K_j) * V_j[d]     (Transformer attention,
 * cited by the paper in Section 1).  K and V are [n][D] row-major.          */
void oracle_attend_unit(const double *q, const double *K, const double *V,
                        int n, int D, double scale, double *out) {
    double *sc = (double *)malloc((size_t)n * sizeof(double));
    double mx = -INFINITY;
    for (int j = 0; j < n; ++j) {
        double s = 0.0;
        for (int d = 0; d < D; ++d) s += q[d] * K[(size_t)j * D + d];
        sc[j] = s * scale;
        if (sc[j] > mx) mx = sc[j];
    }
    double denom = 0.0;
    for (int j = 0; j < n; ++j) {
        sc[j] = exp(sc[j] - mx);
        denom += sc[j];
    }
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    for (int j = 0; j < n; ++j) {
        double p = sc[j] / denom;
        for (int d = 0; d < D; ++d) out[d] += p * V[(size_t)j * D + d];
    }
    free(sc);
}

/* ---- split form of the same sum (rows [j0, j1) only) ---------------------
 * Returns the un-normalised o = sum_j e^{s_j - m} V_j, the block maximum m and
 * l = sum_j e^{s_j - m}.  Together with oracle_combine_partials it restates
 * the softmax sum over a partition of the rows; tests check that any
 * partition reproduces oracle_attend_unit.                                   */
void oracle_partial_unit(const double *q, const double *K, const double *V,
                         int j0, int j1, int D, double scale,
                         double *o, double *m_out, double *l_out) {
    double m = -INFINITY;
    for (int j = j0; j < j1; ++j) {
        double s = 0.0;
        for (int d = 0; d < D; ++d) s += q[d] * K[(size_t)j * D + d];
        s *= scale;
        if (s > m) m = s;
    }
    double l = 0.0;
    for (int d = 0; d < D; ++d) o[d] = 0.0;
    for (int j = j0; j < j1; ++j) {
        double s = 0.0;
        for (int d = 0; d < D; ++d) s += q[d] * K[(size_t)j * D + d];
        double e = exp(s * scale - m);
        l += e;
        for (int d = 0; d < D; ++d) o[d] += e * V[(size_t)j * D + d];
    }
    *m_out = m;
    *l_out = l;
}

/* out = sum_s e^{m_s-M} o_s / sum_s e^{m_s-M} l_s with M = max_s m_s.       */
void oracle_combine_partials(int S, int D, const double *o, const double *m,
                             const double *l, double *out) {
    double M = -INFINITY;
    for (int s = 0; s < S; ++s) if (m[s] > M) M = m[s];
    double denom = 0.0;
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    for (int s = 0; s < S; ++s) {
        double w = exp(m[s] - M);
        denom += w * l[s];
        for (int d = 0; d < D; ++d) out[d] += w * o[(size_t)s * D + d];
    }
    for (int d = 0; d < D; ++d) out[d] /= denom;
}

/* ---- the strategy as a table ---------------------------------------------
 * A layer either computes its own cache or has it replaced by an earlier
 * layer's (Section 3.1: the layer nearer the output is the one replaced).
 * Following replacements back to a layer that computes its own cache gives the
 * layer whose stored K/V the layer really reads; numbering those layers in
 * layer order gives the number of caches that must exist (Table 1, "Layer").
 * Returns the number of distinct computed caches, or -1 for an illegal map.  */
int oracle_slot_table(const int *share_map, int L, int *root_of_layer,
                      int *slot_of_layer) {
    for (int l = 0; l < L; ++l)
        if (share_map[l] < 0 || share_map[l] > l) return -1;
    int n = 0;
    for (int l = 0; l < L; ++l) {
        int r = l;
        while (share_map[r] != r) r = share_map[r];
        root_of_layer[l] = r;
    }
    for (int l = 0; l < L; ++l) {
        if (share_map[l] == l) slot_of_layer[l] = n++;
    }
    for (int l = 0; l < L; ++l) slot_of_layer[l] = slot_of_layer[root_of_layer[l]];
    return n;
}

/* ---- per-layer state ------------------------------------------------------ */
oracle_state *oracle_create(int L, int Hq, int Hkv, int D, int B,
                            const int *share_map, double scale) {
    if (L <= 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || B <= 0) return NULL;
    if (Hq % Hkv != 0) return NULL;
    for (int l = 0; l < L; ++l)
        if (share_map[l] < 0 || share_map[l] > l) return NULL;
    oracle_state *st = (oracle_state *)calloc(1, sizeof(oracle_state));
    st->L = L; st->Hq = Hq; st->Hkv = Hkv; st->D = D; st->B = B;
    st->scale = (scale > 0.0) ? scale : 1.0 / sqrt((double)D);
    st->share_map = (int *)malloc(sizeof(int) * L);
    memcpy(st->share_map, share_map, sizeof(int) * L);
    st->ulen = (int **)calloc(L, sizeof(int *));
    for (int l = 0; l < L; ++l) st->ulen[l] = (int *)calloc((size_t)B * Hkv, sizeof(int));
    st->cap = (int *)calloc(L, sizeof(int));
    st->K = (double ***)calloc(L, sizeof(double **));
    st->V = (double ***)calloc(L, sizeof(double **));
    for (int l = 0; l < L; ++l) {
        st->K[l] = (double **)calloc((size_t)B * Hkv, sizeof(double *));
        st->V[l] = (double **)calloc((size_t)B * Hkv, sizeof(double *));
    }
    return st;
}

void oracle_destroy(oracle_state *st) {
    if (!st) return;
    for (int l = 0; l < st->L; ++l) {
        for (int u = 0; u < st->B * st->Hkv; ++u) { free(st->K[l][u]); free(st->V[l][u]); }
        free(st->K[l]); free(st->V[l]);
    }
    for (int l = 0; l < st->L; ++l) free(st->ulen[l]);
    free(st->K); free(st->V); free(st->ulen); free(st->cap); free(st->share_map);
    free(st);
}

static void ensure_cap(oracle_state *st, int l, int need) {
    if (need <= st->cap[l]) return;
    int nc = st->cap[l] ? st->cap[l] : 16;
    while (nc < need) nc *= 2;
    size_t bytes = (size_t)nc * st->D * sizeof(double);
    for (int u = 0; u < st->B * st->Hkv; ++u) {
        st->K[l][u] = (double *)realloc(st->K[l][u], bytes);
        st->V[l][u] = (double *)realloc(st->V[l][u], bytes);
    }
    st->cap[l] = nc;
}

/* The cache side of one layer's turn in a forward pass (Section 3.2).
 *   layer computes its own cache : append the n_new new rows of
 *       k_new / v_new, laid out [B][n_new][Hkv][D];
 *   layer's cache is replaced    : k_new / v_new are ignored (may be NULL) and
 *       the cache of layer share_map[l], as it stands after that layer's own
 *       turn in this pass, is copied over this layer's cache.
 * Returns 0, or -1 on a bad argument.                                          */
static int max_unit_len(const oracle_state *st, int l) {
    int m = 0;
    for (int u = 0; u < st->B * st->Hkv; ++u) if (st->ulen[l][u] > m) m = st->ulen[l][u];
    return m;
}

static int uniform_len(const oracle_state *st, int l) {   /* common length, or -1 if units differ */
    for (int u = 1; u < st->B * st->Hkv; ++u) if (st->ulen[l][u] != st->ulen[l][0]) return -1;
    return st->ulen[l][0];
}

static int update_cache(oracle_state *st, int l, const double *k_new, const double *v_new, int n_new) {
    const int D = st->D, Hkv = st->Hkv, B = st->B;
    const int src = st->share_map[l];
    if (src == l) {
        if (n_new > 0) {
            if (!k_new || !v_new) return -1;
            ensure_cap(st, l, max_unit_len(st, l) + n_new);
            for (int b = 0; b < B; ++b)
                for (int h = 0; h < Hkv; ++h) {
                    const int u = b * Hkv + h;
                    for (int t = 0; t < n_new; ++t) {
                        size_t in = (((size_t)b * n_new + t) * Hkv + h) * D;
                        size_t row = (size_t)(st->ulen[l][u] + t) * D;
                        memcpy(st->K[l][u] + row, k_new + in, sizeof(double) * D);
                        memcpy(st->V[l][u] + row, v_new + in, sizeof(double) * D);
                    }
                    st->ulen[l][u] += n_new;
                }
        }
    } else {
        /* literal copy of the previously computed layer's cache (sparsified or not) */
        ensure_cap(st, l, max_unit_len(st, src));
        for (int u = 0; u < B * Hkv; ++u) {
            memcpy(st->K[l][u], st->K[src][u], sizeof(double) * (size_t)st->ulen[src][u] * D);
            memcpy(st->V[l][u], st->V[src][u], sizeof(double) * (size_t)st->ulen[src][u] * D);
            st->ulen[l][u] = st->ulen[src][u];
        }
    }
    return 0;
}

/* One layer of one generation step (Section 3.2): the cache update above, then,
 * if q != NULL ([B][Hq][D]), the unchanged attention of the layer's one query
 * per head over the layer's whole cache, written to out ([B][Hq][D]).
 * Returns 0, or -1 on a bad argument / empty cache.                          */
int oracle_layer_forward(oracle_state *st, int l, const double *q,
                         const double *k_new, const double *v_new, int n_new,
                         double *out) {
    if (!st || l < 0 || l >= st->L || n_new < 0) return -1;
    const int D = st->D, Hkv = st->Hkv, Hq = st->Hq, B = st->B;
    if (update_cache(st, l, k_new, v_new, n_new) != 0) return -1;
    if (q) {
        if (!out) return -1;
        for (int u = 0; u < B * Hkv; ++u) if (st->ulen[l][u] <= 0) return -1;
        const int G = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(static)
        for (int b = 0; b < B; ++b)
            for (int hq = 0; hq < Hq; ++hq) {
                int hk = hq / G;
                size_t o = ((size_t)b * Hq + hq) * D;
                oracle_attend_unit(q + o, st->K[l][b * Hkv + hk], st->V[l][b * Hkv + hk],
                                   st->ulen[l][b * Hkv + hk], D, st->scale, out + o);
            }
    }
    return 0;
}

/* One layer of the prefill pass (Section 3.2 applies the strategy to prefill as
 * well as to generation): the same cache update, then n_q queries per head,
 * q [B][n_q][Hq][D], which are the newest n_q positions of the layer's cache.
 * The paper does not restate the mask; decoder models process a prompt with
 * the causal one, so query i (0-based) sees rows 0 .. len - n_q + i and
 * nothing later.  out is [B][n_q][Hq][D].  With n_q = 1 this is
 * oracle_layer_forward.  Returns 0, or -1 on a bad argument.                  */
int oracle_layer_prefill(oracle_state *st, int l, const double *q, int n_q,
                         const double *k_new, const double *v_new, int n_new,
                         double *out) {
    if (!st || l < 0 || l >= st->L || n_new < 0 || n_q < 1 || !q || !out) return -1;
    const int D = st->D, Hkv = st->Hkv, Hq = st->Hq, B = st->B;
    if (update_cache(st, l, k_new, v_new, n_new) != 0) return -1;
    const int n = uniform_len(st, l);   /* positions are only defined while no rows were evicted */
    if (n < 0 || n_q > n) return -1;
    const int G = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < n_q; ++i)
            for (int hq = 0; hq < Hq; ++hq) {
                int hk = hq / G;
                size_t o = (((size_t)b * n_q + i) * Hq + hq) * D;
                oracle_attend_unit(q + o, st->K[l][b * Hkv + hk], st->V[l][b * Hkv + hk],
                                   n - n_q + i + 1, D, st->scale, out + o);
            }
    return 0;
}

/* Longest (sequence, head) of layer l's cache (all are equal unless rows were evicted). */
int oracle_len(const oracle_state *st, int l) {
    return (st && l >= 0 && l < st->L) ? max_unit_len(st, l) : -1;
}

int oracle_unit_len(const oracle_state *st, int l, int b, int h) {
    if (!st || l < 0 || l >= st->L || b < 0 || b >= st->B || h < 0 || h >= st->Hkv) return -1;
    return st->ulen[l][b * st->Hkv + h];
}

/* Intra-layer compression applied to a layer that computes its own cache (Section 4.4 and the
 * reproduction appendix: each layer's cache is sparsified in turn by H2O / PyramidInfer, and
 * a layer that shares receives the sparsified cache of its source, which here happens by the
 * usual literal copy at the sharing layer's next turn).  Which rows survive is the outside
 * method's decision: keep[(b*Hkv+h)*keep_stride + j], j < n_keep[b*Hkv+h], strictly ascending
 * row indices of unit (b,h).  The kept rows move to the front in order; the rest is gone.
 * Returns 0, or -1 for a sharing layer, an empty or non-ascending or out-of-range list.      */
int oracle_evict(oracle_state *st, int l, const int *keep, const int *n_keep, int keep_stride) {
    if (!st || l < 0 || l >= st->L || !keep || !n_keep || st->share_map[l] != l) return -1;
    const int D = st->D;
    for (int u = 0; u < st->B * st->Hkv; ++u) {
        if (n_keep[u] < 1 || n_keep[u] > st->ulen[l][u] || n_keep[u] > keep_stride) return -1;
        for (int j = 0; j < n_keep[u]; ++j) {
            int r = keep[(size_t)u * keep_stride + j];
            if (r < 0 || r >= st->ulen[l][u] || (j > 0 && r <= keep[(size_t)u * keep_stride + j - 1])) return -1;
        }
    }
    for (int u = 0; u < st->B * st->Hkv; ++u) {
        for (int j = 0; j < n_keep[u]; ++j) {
            int r = keep[(size_t)u * keep_stride + j];
            memmove(st->K[l][u] + (size_t)j * D, st->K[l][u] + (size_t)r * D, sizeof(double) * D);
            memmove(st->V[l][u] + (size_t)j * D, st->V[l][u] + (size_t)r * D, sizeof(double) * D);
        }
        st->ulen[l][u] = n_keep[u];
    }
    return 0;
}

/* Copy layer l's cache out as [B][Hkv][len][D] with len = oracle_len (K then V into
 * separate buffers; rows past a unit's own length are zero), for bit-exact comparison
 * with what the GPU pool holds.                                               */
int oracle_get_cache(const oracle_state *st, int l, double *K_out, double *V_out) {
    if (!st || l < 0 || l >= st->L) return -1;
    const int n = max_unit_len(st, l);
    size_t rows = (size_t)n * st->D;
    for (int u = 0; u < st->B * st->Hkv; ++u) {
        size_t have = (size_t)st->ulen[l][u] * st->D;
        memcpy(K_out + u * rows, st->K[l][u], sizeof(double) * have);
        memcpy(V_out + u * rows, st->V[l][u], sizeof(double) * have);
        memset(K_out + u * rows + have, 0, sizeof(double) * (rows - have));
        memset(V_out + u * rows + have, 0, sizeof(double) * (rows - have));
    }
    return 0;
}

/* ---- the data-parallel part of strategy searching (Section 3.1) --------------
 * Similarity of KV caches: the cache of every layer is averaged over the calibration
 * samples (here: over the B sequences held), keys and values are each flattened,
 * and the Euclidean distance between the representations of any two layers is
 * taken.  The averaging step of Section 3.1 / Algorithm 1 can be read in more than
 * one way (keys and values are to be averaged apart from each other); reading: the
 * representation of a layer is the sample-mean of its keys, flattened, followed by
 * the sample-mean of its values, flattened; the distance is the 2-norm of the
 * difference of two such vectors.  All layers must hold equally long, un-evicted
 * caches.  dist is [L][L], symmetric, zero diagonal.  Returns 0 or -1.          */
int oracle_layer_distances(const oracle_state *st, double *dist) {
    if (!st || !dist) return -1;
    const int L = st->L, U = st->B * st->Hkv, B = st->B, Hkv = st->Hkv, D = st->D;
    const int n = uniform_len(st, 0);
    if (n <= 0) return -1;
    for (int l = 1; l < L; ++l) if (uniform_len(st, l) != n) return -1;
    (void)U;
    const size_t P = (size_t)Hkv * n * D;            /* elements of one flattened K (or V) */
    double *rep = (double *)calloc((size_t)L * 2 * P, sizeof(double));
    for (int l = 0; l < L; ++l)
        for (int h = 0; h < Hkv; ++h)
            for (size_t e = 0; e < (size_t)n * D; ++e) {
                double sk = 0.0, sv = 0.0;
                for (int b = 0; b < B; ++b) {
                    sk += st->K[l][b * Hkv + h][e];
                    sv += st->V[l][b * Hkv + h][e];
                }
                rep[((size_t)l * 2 + 0) * P + (size_t)h * n * D + e] = sk / B;
                rep[((size_t)l * 2 + 1) * P + (size_t)h * n * D + e] = sv / B;
            }
    for (int i = 0; i < L; ++i)
        for (int j = 0; j < L; ++j) {
            double s = 0.0;
            for (size_t e = 0; e < 2 * P; ++e) {
                double d = rep[(size_t)i * 2 * P + e] - rep[(size_t)j * 2 * P + e];
                s += d * d;
            }
            dist[(size_t)i * L + j] = sqrt(s);
        }
    free(rep);
    return 0;
}

/* "Avg_Cos_Sim" (Algorithm 1, Section 3.1): the last-layer output representations of
 * two models on the calibration sentences, a and b, each [S][dim], are averaged over the
 * S sentences and the cosine similarity of the two averaged vectors is returned.        */
double oracle_mean_cosine(const double *a, const double *b, int S, long long dim) {
    double dot = 0.0, na = 0.0, nb = 0.0;
    for (long long e = 0; e < dim; ++e) {
        double ma = 0.0, mb = 0.0;
        for (int s = 0; s < S; ++s) {
            ma += a[(size_t)s * dim + e];
            mb += b[(size_t)s * dim + e];
        }
        ma /= S; mb /= S;
        dot += ma * mb; na += ma * ma; nb += mb * mb;
    }
    return dot / (sqrt(na) * sqrt(nb));
}

/* Many independent units at once (the benchmark's CPU-baseline leg and the
 * sampled-unit parity checks at sizes the stateful oracle cannot hold):
 * unit u has query q[u][D], keys K[u][n][D], values V[u][n][D].              */
void oracle_attend_units(const double *q, const double *K, const double *V,
                         int units, int n, int D, double scale, double *out) {
#pragma omp parallel for schedule(static)
    for (int u = 0; u < units; ++u)
        oracle_attend_unit(q + (size_t)u * D, K + (size_t)u * n * D,
                           V + (size_t)u * n * D, n, D, scale, out + (size_t)u * D);
}
