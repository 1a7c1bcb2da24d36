/*
 * CPU oracle for the HAC / sHAC formats and their compressed-domain product.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference the CUDA
 * library is checked against.  It shares no code with that library and is
 * never called by it.  All floating point is IEEE fp64, accumulated in the
 * order the paper's procedures state; build with -ffp-contract=off and
 * without fast-math.
 *
 * What each routine follows (Marino, Petrini, Malchiodi, Frasca, "Compact
 * representations of convolutional neural networks via weight pruning and
 * quantization"):
 *   orc_kmeans            Sect. III-C.1 (CWS: k-means on the weights)
 *   orc_pack              Sect. IV-B (HAC bit stream split into b = 32 bit
 *                         words, zero padding of the last word)
 *   orc_dot_hac           Algorithm 1 (Dot_HAC) with the NCW procedure
 *   orc_dot_shac          Algorithm 2 (Dot_sHAC)
 *   orc_pardot_*          Algorithm 3 (ParDot: rows of X split over q threads)
 *   orc_dot_definition    the plain definition x^T W the algorithms output
 *   orc_decode            inverse of orc_pack (the formats are lossless)
 *
 * Indices are 0-based here; the paper's are 1-based.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>
#include <pthread.h>

/* ------------------------------------------------------------------------- */
/* Sect. III-C.1: k-means on a list of scalars (Lloyd iterations).            */
/*                                                                            */
/* data[q]     the non-null weights, in the order they are stored (by column) */
/* c[k]        in: initial centroids, ascending; out: final centroids         */
/* assign[q]   out: cluster of every weight under the final centroids         */
/* sse[iters+1] out: sum of squared distances to the assigned centroid before */
/*             every update and after the last one (for the tests)            */
/*                                                                            */
/* Assignment: with centroids sorted ascending, the nearest centroid of w is  */
/* found from the midpoints t_l = (c_l + c_{l+1}) / 2: cluster = number of    */
/* midpoints strictly below w (a weight equal to a midpoint goes down).       */
/* Update: c_l = mean of its cluster, sums taken sequentially in storage      */
/* order; an empty cluster keeps its centroid; centroids are then re-sorted.  */
/* ------------------------------------------------------------------------- */
static int cmp_double(const void* a, const void* b) {
    double x = *(const double*)a, y = *(const double*)b;
    return (x > y) - (x < y);
}

static int32_t cluster_of(double w, const double* t, int32_t k) {
    /* number of midpoints t[0..k-2] that are < w  (binary search) */
    int32_t lo = 0, hi = k - 1;
    while (lo < hi) {
        int32_t mid = (lo + hi) / 2;
        if (t[mid] < w) lo = mid + 1; else hi = mid;
    }
    return lo;
}

int orc_kmeans(const double* data, int64_t q, double* c, int32_t k, int32_t iters,
               int32_t* assign, double* sse) {
    if (k < 1 || q < 1) return -1;
    double* t = (double*)malloc(sizeof(double) * (size_t)(k > 1 ? k - 1 : 1));
    double* sum = (double*)malloc(sizeof(double) * (size_t)k);
    int64_t* cnt = (int64_t*)malloc(sizeof(int64_t) * (size_t)k);
    if (!t || !sum || !cnt) return -2;
    for (int32_t it = 0; it <= iters; ++it) {
        for (int32_t l = 0; l + 1 < k; ++l) t[l] = (c[l] + c[l + 1]) * 0.5;
        for (int32_t l = 0; l < k; ++l) { sum[l] = 0.0; cnt[l] = 0; }
        double e = 0.0;
        for (int64_t p = 0; p < q; ++p) {
            int32_t l = cluster_of(data[p], t, k);
            assign[p] = l;
            sum[l] += data[p];
            cnt[l] += 1;
            double d = data[p] - c[l];
            e += d * d;
        }
        if (sse) sse[it] = e;
        if (it == iters) break;              /* last pass only assigns */
        for (int32_t l = 0; l < k; ++l)
            if (cnt[l] > 0) c[l] = sum[l] / (double)cnt[l];
        qsort(c, (size_t)k, sizeof(double), cmp_double);
    }
    free(t); free(sum); free(cnt);
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Sect. IV-B: concatenate the code words of a symbol sequence, first bit of  */
/* the stream in the most significant bit of word 0, N = ceil(bits / 32)      */
/* words, the last one padded with zero bits.  Written one bit at a time.     */
/*   sym[count]       symbol ids in stream order                              */
/*   code[k], len[k]  code word of every symbol (value and bit length)        */
/*   words[nwords]    out (caller allocates ceil(total_bits/32), zero-filled) */
/* returns the number of bits written, or -1 if words[] is too short          */
/* ------------------------------------------------------------------------- */
int64_t orc_pack(const int32_t* sym, int64_t count, const uint32_t* code, const uint8_t* len,
                 uint32_t* words, int64_t nwords) {
    int64_t bit = 0;
    for (int64_t p = 0; p < count; ++p) {
        uint32_t cw = code[sym[p]];
        int l = len[sym[p]];
        for (int b = l - 1; b >= 0; --b) {
            if ((bit >> 5) >= nwords) return -1;
            if ((cw >> b) & 1u) words[bit >> 5] |= (uint32_t)1 << (31 - (bit & 31));
            ++bit;
        }
    }
    return bit;
}

/* ------------------------------------------------------------------------- */
/* Decoding dictionary H^{-1} as an explicit binary tree.                     */
/* node 0 is the root; child[2*v + bit] is the next node or -1; leaf[v] is    */
/* the symbol id at a leaf, -1 inside the tree.                               */
/* ------------------------------------------------------------------------- */
typedef struct {
    int32_t* child;
    int32_t* leaf;
    int32_t nodes;
} orc_tree;

static int tree_build(orc_tree* T, const uint32_t* code, const uint8_t* len, int32_t k) {
    int64_t cap = 1;
    for (int32_t s = 0; s < k; ++s) cap += len[s];
    T->child = (int32_t*)malloc(sizeof(int32_t) * 2 * (size_t)cap);
    T->leaf = (int32_t*)malloc(sizeof(int32_t) * (size_t)cap);
    if (!T->child || !T->leaf) return -2;
    for (int64_t v = 0; v < cap; ++v) { T->child[2 * v] = T->child[2 * v + 1] = -1; T->leaf[v] = -1; }
    T->nodes = 1;
    for (int32_t s = 0; s < k; ++s) {
        int32_t v = 0;
        for (int b = len[s] - 1; b >= 0; --b) {
            int bit = (int)((code[s] >> b) & 1u);
            if (T->leaf[v] >= 0) return -3;            /* not a prefix code */
            if (T->child[2 * v + bit] < 0) T->child[2 * v + bit] = T->nodes++;
            v = T->child[2 * v + bit];
        }
        if (T->leaf[v] >= 0 || T->child[2 * v] >= 0 || T->child[2 * v + 1] >= 0) return -3;
        T->leaf[v] = s;
    }
    return 0;
}

static void tree_free(orc_tree* T) { free(T->child); free(T->leaf); }

/* getBinarySeq of Algorithms 1 and 2: the 32 bits of one word, first bit first. */
static void get_binary_seq(uint32_t word, uint8_t S[32]) {
    for (int b = 0; b < 32; ++b) S[b] = (uint8_t)((word >> (31 - b)) & 1u);
}

/* NCW (next code word), Sect. IV-B.  Scans S from position *oset.  *rem is
 * the tree node reached by the bits of an unfinished code word carried over
 * from the previous memory word (0 = root = nothing carried).  Returns 1 and
 * the symbol in *z when a code word ends inside S; returns 0 ("null") when S
 * is exhausted first, leaving the partial code word in *rem and *oset = 0. */
static int ncw(const orc_tree* T, const uint8_t S[32], int32_t* rem, int* oset, int32_t* z) {
    int32_t v = *rem;
    int o = *oset;
    while (o < 32) {
        v = T->child[2 * v + S[o]];
        ++o;
        if (v < 0) return -1;                    /* bits that are no code word: corrupt stream */
        if (T->leaf[v] >= 0) { *z = T->leaf[v]; *rem = 0; *oset = o; return 1; }
    }
    *rem = v; *oset = 0;
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Algorithm 1, Dot_HAC.  out has one entry per column (m of them).  The scan */
/* stops after n*m symbols: a run of zero bits is a valid code word of a      */
/* complete code, so only the count tells padding from data.                  */
/* ------------------------------------------------------------------------- */
static int dot_hac_tree(const uint32_t* C, int64_t N, const orc_tree* T, const float* value,
                        const float* x, int64_t n, int64_t m, double* out) {
    int64_t row = 0, col = 0, total = n * m, done = 0;
    double sum = 0.0;
    int32_t rem = 0, z = 0;
    int oset = 0;
    for (int64_t j = 0; j < m; ++j) out[j] = 0.0;
    for (int64_t i = 0; i < N && done < total; ++i) {
        uint8_t S[32];
        get_binary_seq(C[i], S);
        int r;
        while (done < total && (r = ncw(T, S, &rem, &oset, &z)) != 0) {
            if (r < 0) return -4;
            sum = sum + (double)x[row] * (double)value[z];
            row = row + 1;
            ++done;
            if (row >= n) {
                row = 0; out[col] = sum;
                col = col + 1; sum = 0.0;
            }
        }
    }
    return done == total ? 0 : -5;
}

int orc_dot_hac(const uint32_t* C, int64_t N, const uint32_t* code, const uint8_t* len,
                const float* value, int32_t k, const float* x, int64_t n, int64_t m, double* out) {
    orc_tree T;
    int rc = tree_build(&T, code, len, k);
    if (rc == 0) rc = dot_hac_tree(C, N, &T, value, x, n, m, out);
    tree_free(&T);
    return rc;
}

/* ------------------------------------------------------------------------- */
/* Algorithm 2, Dot_sHAC.  pos walks nz; columns whose cb entries coincide    */
/* are empty and skipped; their outputs stay at the initial zero.             */
/* ------------------------------------------------------------------------- */
static int dot_shac_tree(const uint32_t* C, int64_t N1, const orc_tree* T, const float* value,
                         const int32_t* ri, const int64_t* cb, const float* x, int64_t m,
                         double* out) {
    int64_t pos = 0, col = 0, q = cb[m];
    double sum = 0.0;
    int32_t rem = 0, z = 0;
    int oset = 0;
    for (int64_t j = 0; j < m; ++j) out[j] = 0.0;
    for (int64_t i = 0; i < N1 && pos < q; ++i) {
        uint8_t S[32];
        get_binary_seq(C[i], S);
        int r;
        while (pos < q && (r = ncw(T, S, &rem, &oset, &z)) != 0) {
            if (r < 0) return -4;
            while (cb[col + 1] == pos) col = col + 1;       /* skip empty columns */
            sum = sum + (double)x[ri[pos]] * (double)value[z];
            pos = pos + 1;
            if (cb[col + 1] == pos) {
                out[col] = sum;
                sum = 0.0; col = col + 1;
            }
        }
    }
    return pos == q ? 0 : -5;
}

int orc_dot_shac(const uint32_t* C, int64_t N1, const uint32_t* code, const uint8_t* len,
                 const float* value, int32_t k, const int32_t* ri, const int64_t* cb,
                 const float* x, int64_t m, double* out) {
    orc_tree T;
    int rc = tree_build(&T, code, len, k);
    if (rc == 0) rc = dot_shac_tree(C, N1, &T, value, ri, cb, x, m, out);
    tree_free(&T);
    return rc;
}

/* ------------------------------------------------------------------------- */
/* Algorithm 3, ParDot.  X is B x n (one input per row), out is B x m.  The   */
/* rows are cut into q chunks of ceil(B/q); every computing unit runs the     */
/* sequential Dot procedure once per row of its chunk.                        */
/* ------------------------------------------------------------------------- */
typedef struct {
    int shac;
    const uint32_t* C; int64_t N; const orc_tree* T; const float* value;
    const int32_t* ri; const int64_t* cb;
    const float* X; int64_t n, m; double* out;
    int64_t start, end;
    int rc;
} pardot_job;

static void* pardot_worker(void* arg) {
    pardot_job* J = (pardot_job*)arg;
    J->rc = 0;
    for (int64_t i = J->start; i < J->end; ++i) {
        const float* x = J->X + i * J->n;
        double* y = J->out + i * J->m;
        int rc = J->shac ? dot_shac_tree(J->C, J->N, J->T, J->value, J->ri, J->cb, x, J->m, y)
                         : dot_hac_tree(J->C, J->N, J->T, J->value, x, J->n, J->m, y);
        if (rc) J->rc = rc;
    }
    return NULL;
}

static int pardot(int shac, const uint32_t* C, int64_t N, const uint32_t* code, const uint8_t* len,
                  const float* value, int32_t k, const int32_t* ri, const int64_t* cb,
                  const float* X, int64_t B, int64_t n, int64_t m, int32_t q, double* out) {
    if (q < 1) return -1;
    orc_tree T;
    int rc = tree_build(&T, code, len, k);
    if (rc) { tree_free(&T); return rc; }
    int64_t chunk = (B + q - 1) / q;
    pthread_t* th = (pthread_t*)malloc(sizeof(pthread_t) * (size_t)q);
    pardot_job* job = (pardot_job*)malloc(sizeof(pardot_job) * (size_t)q);
    int32_t started = 0;
    for (int32_t u = 0; u < q; ++u) {
        int64_t s = u * chunk, e = s + chunk;
        if (e > B) e = B;
        if (s >= e) break;
        pardot_job J = { shac, C, N, &T, value, ri, cb, X, n, m, out, s, e, 0 };
        job[u] = J;
        pthread_create(&th[u], NULL, pardot_worker, &job[u]);
        ++started;
    }
    for (int32_t u = 0; u < started; ++u) { pthread_join(th[u], NULL); if (job[u].rc) rc = job[u].rc; }
    free(th); free(job); tree_free(&T);
    return rc;
}

int orc_pardot_hac(const uint32_t* C, int64_t N, const uint32_t* code, const uint8_t* len,
                   const float* value, int32_t k, const float* X, int64_t B, int64_t n, int64_t m,
                   int32_t q, double* out) {
    return pardot(0, C, N, code, len, value, k, NULL, NULL, X, B, n, m, q, out);
}

int orc_pardot_shac(const uint32_t* C, int64_t N1, const uint32_t* code, const uint8_t* len,
                    const float* value, int32_t k, const int32_t* ri, const int64_t* cb,
                    const float* X, int64_t B, int64_t n, int64_t m, int32_t q, double* out) {
    return pardot(1, C, N1, code, len, value, k, ri, cb, X, B, n, m, q, out);
}

/* ------------------------------------------------------------------------- */
/* The plain definition of what Algorithms 1-3 output:                        */
/*   y[b][j] = sum_{i=0}^{n-1} Wq[i][j] * X[b][i]        (i ascending, fp64)  */
/*   a[b][j] = sum_i |Wq[i][j] * X[b][i]|                (tolerance scale)    */
/* Wq is n x m row-major fp32.                                                */
/* ------------------------------------------------------------------------- */
int orc_dot_definition(const float* Wq, int64_t n, int64_t m, const float* X, int64_t B,
                       double* y, double* a) {
    for (int64_t b = 0; b < B; ++b)
        for (int64_t j = 0; j < m; ++j) {
            double s = 0.0, t = 0.0;
            for (int64_t i = 0; i < n; ++i) {
                double p = (double)Wq[i * m + j] * (double)X[b * n + i];
                s = s + p;
                t = t + fabs(p);
            }
            y[b * m + j] = s;
            if (a) a[b * m + j] = t;
        }
    return 0;
}

/* The same definition for selected outputs only (full-size spot checks):
 * cols[c] is evaluated for every input row b; y and a are B x ncols.      */
int orc_dot_definition_cols(const float* Wq, int64_t n, int64_t m, const float* X, int64_t B,
                            const int64_t* cols, int64_t ncols, double* y, double* a) {
    for (int64_t b = 0; b < B; ++b)
        for (int64_t c = 0; c < ncols; ++c) {
            int64_t j = cols[c];
            if (j < 0 || j >= m) return -1;
            double s = 0.0, t = 0.0;
            for (int64_t i = 0; i < n; ++i) {
                double p = (double)Wq[i * m + j] * (double)X[b * n + i];
                s = s + p;
                t = t + fabs(p);
            }
            y[b * ncols + c] = s;
            if (a) a[b * ncols + c] = t;
        }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Inverse of orc_pack: read `count` symbols from the stream, starting at bit */
/* `bit0`, by walking the tree one bit at a time.  Returns the bit position   */
/* after the last symbol, or a negative error.                                */
/* ------------------------------------------------------------------------- */
int64_t orc_decode(const uint32_t* words, int64_t nwords, int64_t bit0, const uint32_t* code,
                   const uint8_t* len, int32_t k, int64_t count, int32_t* sym_out) {
    orc_tree T;
    int rc = tree_build(&T, code, len, k);
    if (rc) { tree_free(&T); return rc; }
    int64_t bit = bit0;
    for (int64_t p = 0; p < count; ++p) {
        int32_t v = 0;
        while (T.leaf[v] < 0) {
            if ((bit >> 5) >= nwords) { tree_free(&T); return -6; }
            int b = (int)((words[bit >> 5] >> (31 - (bit & 31))) & 1u);
            v = T.child[2 * v + b];
            ++bit;
            if (v < 0) { tree_free(&T); return -4; }
        }
        sym_out[p] = T.leaf[v];
    }
    tree_free(&T);
    return bit;
}
