/*
 * CPU ORACLE for the thresholded all-pairs similarity join.
 *
 * THIS FILE IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the tests, the
 * smoke check and the benchmark's cpu_baseline / reference legs may build,
 * load or call it.  It shares no code, header, table or constant with the CUDA
 * library and includes nothing from it.
 *
 * What it computes: the definition of the similarity join in Section 4 of the
 * paper (P join_r Q = all pairs (x, y) in P x Q whose distance is at most r),
 * taken over index pairs (i, j), for the ip-distances Section 4 lists, written
 * as the plain double loop over (i, j) with an inner loop over the d
 * coordinates.  The paper's brute-force TCU algorithm (Section 4, the product
 * F_P * G_Q^T evaluated with Theorem 1's tiling) reaches exactly this set, so
 * the definition itself is the oracle: no tiling, blocking or reordering here.
 *
 * Readings where the paper is silent (each one is listed in the design notes):
 *   - similarities (inner product, cosine) pass when score >= t, distances
 *     (Euclidean) when distance <= r; both inclusive, as "D(x,y) <= r" is.
 *   - points are identified by their row index; duplicates are distinct rows;
 *     a self join keeps the diagonal and both orientations.
 *   - int8 inputs: exact integer arithmetic.  Inner product: pass iff
 *     s >= t over the reals (s is an integer below 2^53, so the double compare
 *     is exact).  Euclidean: pass iff the integer squared distance D satisfies
 *     (double)D <= r*r, r*r being the double product.  Cosine: the three sums
 *     <x,y>, |x|^2, |y|^2 and the product |x|^2 |y|^2 are exact integers;
 *     the score is the fp64 quotient <x,y> / sqrt(|x|^2 |y|^2) (conversion of
 *     the product to double, IEEE sqrt, IEEE quotient: three roundings), 0 for
 *     a zero vector; pass iff score >= t.  The score is a floating-point number
 *     that decides an integer result, so this exact sequence is part of the
 *     reading; with it parallel rows score exactly 1.
 *   - bf16 inputs: the 16-bit patterns are the inputs; each is widened exactly
 *     to fp64 and all sums run in fp64 with k ascending.
 *     cosine of a zero vector is defined as 0.
 *     Euclidean uses the difference form sqrt(sum (x_k-y_k)^2), not the norm
 *     expansion.
 *
 * Output: pairs sorted by (i, j); the return value is the total number of
 * passing pairs even when it exceeds `capacity` (then only the first
 * `capacity` pairs in sorted order are written).  -1 on invalid arguments.
 *
 * Threads only split the outer loop into contiguous row blocks whose results
 * are concatenated in block order; they do not change any arithmetic.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { KIND_IP = 0, KIND_COS = 1, KIND_L2 = 2 };

/* ---------------------------------------------------------------- scores */

/* <x,y> over int8 coordinates, exact. */
int64_t oracle_ip_i8(const int8_t *x, const int8_t *y, int32_t d) {
    int64_t s = 0;
    for (int32_t k = 0; k < d; ++k) s += (int64_t)x[k] * (int64_t)y[k];
    return s;
}

/* sum_k (x_k - y_k)^2 over int8 coordinates, exact. */
int64_t oracle_sqdist_i8(const int8_t *x, const int8_t *y, int32_t d) {
    int64_t s = 0;
    for (int32_t k = 0; k < d; ++k) {
        int64_t e = (int64_t)x[k] - (int64_t)y[k];
        s += e * e;
    }
    return s;
}

/* Cosine of two int8 rows: <x,y>, |x|^2 and |y|^2 as exact integers, their product |x|^2 |y|^2 as an exact
 * 64-bit integer (below 2^63 for rows of up to 2^17 coordinates), then three fp64 roundings: the integer to
 * double, the square root, the quotient.  Parallel rows score exactly 1: the product is then a perfect square. */
double oracle_cos_i8(const int8_t *x, const int8_t *y, int32_t d) {
    int64_t s = oracle_ip_i8(x, y, d), nx = oracle_ip_i8(x, x, d), ny = oracle_ip_i8(y, y, d);
    if (nx == 0 || ny == 0) return 0.0;
    return (double)s / sqrt((double)(nx * ny));
}

/* The value a bfloat16 bit pattern denotes, as fp64 (exact). */
double oracle_bf16_to_f64(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static double dot_f64(const double *x, const double *y, int32_t d) {
    double s = 0.0;
    for (int32_t k = 0; k < d; ++k) s += x[k] * y[k];
    return s;
}

/* Score of one pair of already widened rows; nx2, ny2 are sum x_k^2, sum y_k^2
 * (used by the cosine only). */
static double score_f64(const double *x, const double *y, int32_t d, int kind, double nx2, double ny2) {
    if (kind == KIND_IP) return dot_f64(x, y, d);
    if (kind == KIND_COS) {
        if (nx2 == 0.0 || ny2 == 0.0) return 0.0;
        return dot_f64(x, y, d) / (sqrt(nx2) * sqrt(ny2));
    }
    double s = 0.0;
    for (int32_t k = 0; k < d; ++k) {
        double e = x[k] - y[k];
        s += e * e;
    }
    return sqrt(s);
}

static double *widen_rows(const uint16_t *X, int64_t rows, int32_t d) {
    size_t cnt = (size_t)rows * (size_t)d;
    double *W = (double *)malloc((cnt ? cnt : 1) * sizeof(double));
    if (!W) return NULL;
    for (size_t t = 0; t < cnt; ++t) W[t] = oracle_bf16_to_f64(X[t]);
    return W;
}

static double *row_sq_norms(const double *W, int64_t rows, int32_t d) {
    double *N = (double *)malloc((rows ? rows : 1) * sizeof(double));
    if (!N) return NULL;
    for (int64_t i = 0; i < rows; ++i) N[i] = dot_f64(W + (size_t)i * d, W + (size_t)i * d, d);
    return N;
}

/* Score of the bf16 pair (row i of P, row j of Q), fp64. */
double oracle_score_bf16(const uint16_t *P, int64_t i, const uint16_t *Q, int64_t j, int32_t d, int32_t kind) {
    double *x = widen_rows(P + (size_t)i * d, 1, d);
    double *y = widen_rows(Q + (size_t)j * d, 1, d);
    double s = score_f64(x, y, d, kind, dot_f64(x, x, d), dot_f64(y, y, d));
    free(x);
    free(y);
    return s;
}

/* Scores of a list of pairs: out[p] = score(P[pairs[2p]], Q[pairs[2p+1]]).
 * int8: inner product (KIND_IP) or squared distance (KIND_L2) as int64 in out_i, cosine as fp64
 * (oracle_scores_cos_i8); bf16: fp64 score in out_f. */
int32_t oracle_scores_i8(const int8_t *P, const int8_t *Q, int32_t d, int32_t kind,
                         const int32_t *pairs, int64_t npairs, int64_t *out_i) {
    if (kind != KIND_IP && kind != KIND_L2) return -1;
    for (int64_t p = 0; p < npairs; ++p) {
        const int8_t *x = P + (size_t)pairs[2 * p] * d, *y = Q + (size_t)pairs[2 * p + 1] * d;
        out_i[p] = kind == KIND_IP ? oracle_ip_i8(x, y, d) : oracle_sqdist_i8(x, y, d);
    }
    return 0;
}

int32_t oracle_scores_cos_i8(const int8_t *P, const int8_t *Q, int32_t d, const int32_t *pairs, int64_t npairs, double *out_f) {
    for (int64_t p = 0; p < npairs; ++p)
        out_f[p] = oracle_cos_i8(P + (size_t)pairs[2 * p] * d, Q + (size_t)pairs[2 * p + 1] * d, d);
    return 0;
}

int32_t oracle_scores_bf16(const uint16_t *P, const uint16_t *Q, int32_t d, int32_t kind,
                           const int32_t *pairs, int64_t npairs, double *out_f) {
    if (kind < KIND_IP || kind > KIND_L2) return -1;
    for (int64_t p = 0; p < npairs; ++p)
        out_f[p] = oracle_score_bf16(P, pairs[2 * p], Q, pairs[2 * p + 1], d, kind);
    return 0;
}

/* Row squared norms in fp64 (bf16 rows) / exact int64 (int8 rows). */
void oracle_sq_norms_bf16(const uint16_t *X, int64_t rows, int32_t d, double *out) {
    for (int64_t i = 0; i < rows; ++i) {
        double s = 0.0;
        for (int32_t k = 0; k < d; ++k) {
            double v = oracle_bf16_to_f64(X[(size_t)i * d + k]);
            s += v * v;
        }
        out[i] = s;
    }
}

void oracle_sq_norms_i8(const int8_t *X, int64_t rows, int32_t d, int64_t *out) {
    for (int64_t i = 0; i < rows; ++i) out[i] = oracle_ip_i8(X + (size_t)i * d, X + (size_t)i * d, d);
}

/* ------------------------------------------------------------- the join */

typedef struct {
    int32_t *v;     /* (i, j) pairs of this row block, in (i, j) order */
    int64_t cnt, cap;
    int oom;
} pairbuf;

static void pb_push(pairbuf *b, int64_t i, int64_t j) {
    if (b->cnt == b->cap) {
        int64_t nc = b->cap ? 2 * b->cap : 64;
        int32_t *nv = (int32_t *)realloc(b->v, (size_t)nc * 2 * sizeof(int32_t));
        if (!nv) { b->oom = 1; return; }
        b->v = nv;
        b->cap = nc;
    }
    b->v[2 * b->cnt] = (int32_t)i;
    b->v[2 * b->cnt + 1] = (int32_t)j;
    b->cnt++;
}

static int pass_i8(const int8_t *x, const int8_t *y, int32_t d, int kind, double thr) {
    if (kind == KIND_IP) return (double)oracle_ip_i8(x, y, d) >= thr;
    if (kind == KIND_COS) return oracle_cos_i8(x, y, d) >= thr;
    return (double)oracle_sqdist_i8(x, y, d) <= thr * thr;
}

static int pass_f64(double score, int kind, double thr) {
    return kind == KIND_L2 ? score <= thr : score >= thr;
}

static int64_t num_blocks(int64_t n, int nthreads) {
    int64_t nb = (int64_t)nthreads * 64;
    if (nb > n) nb = n;
    if (nb < 1) nb = 1;
    return nb;
}

static int64_t gather(pairbuf *blk, int64_t nb, int32_t *out_pairs, int64_t capacity) {
    int64_t total = 0, written = 0;
    int oom = 0;
    for (int64_t b = 0; b < nb; ++b) {
        oom |= blk[b].oom;
        for (int64_t p = 0; p < blk[b].cnt && written < capacity; ++p, ++written) {
            out_pairs[2 * written] = blk[b].v[2 * p];
            out_pairs[2 * written + 1] = blk[b].v[2 * p + 1];
        }
        total += blk[b].cnt;
        free(blk[b].v);
    }
    free(blk);
    return oom ? -1 : total;
}

static int resolve_threads(int32_t nthreads) {
#ifdef _OPENMP
    return nthreads > 0 ? nthreads : omp_get_max_threads();
#else
    (void)nthreads;
    return 1;
#endif
}

int32_t oracle_max_threads(void) { return resolve_threads(0); }

int64_t oracle_join_i8(const int8_t *P, int64_t n, const int8_t *Q, int64_t m, int32_t d, int32_t kind,
                       double threshold, int32_t *out_pairs, int64_t capacity, int32_t nthreads) {
    if (n < 0 || m < 0 || d <= 0 || capacity < 0 || kind < KIND_IP || kind > KIND_L2) return -1;
    if (isnan(threshold) || (kind == KIND_L2 && threshold < 0)) return -1;
    if (n >= INT32_MAX || m >= INT32_MAX) return -1;
    int nt = resolve_threads(nthreads);
    int64_t nb = num_blocks(n, nt);
    pairbuf *blk = (pairbuf *)calloc((size_t)nb, sizeof(pairbuf));
    if (!blk) return -1;
#pragma omp parallel for schedule(dynamic, 1) num_threads(nt)
    for (int64_t b = 0; b < nb; ++b) {
        int64_t i0 = n * b / nb, i1 = n * (b + 1) / nb;
        for (int64_t i = i0; i < i1; ++i)
            for (int64_t j = 0; j < m; ++j)
                if (pass_i8(P + (size_t)i * d, Q + (size_t)j * d, d, kind, threshold)) pb_push(&blk[b], i, j);
    }
    return gather(blk, nb, out_pairs, capacity);
}

/* Hamming distance of two bit-packed rows of d coordinates (d/8 bytes each; coordinate k is bit
 * k%8 of byte k/8): the number of coordinates that differ -- Section 4's first ip-distance. */
int64_t oracle_hamming_bits(const uint8_t *x, const uint8_t *y, int32_t d) {
    int64_t h = 0;
    for (int32_t k = 0; k < d; ++k) {
        int bx = (x[k >> 3] >> (k & 7)) & 1, by = (y[k >> 3] >> (k & 7)) & 1;
        h += bx != by;
    }
    return h;
}

/* All (i, j) with Hamming(P[i], Q[j]) <= r over bit-packed rows; output as in the other joins. */
int64_t oracle_join_hamming_bits(const uint8_t *P, int64_t n, const uint8_t *Q, int64_t m, int32_t d, double r,
                                 int32_t *out_pairs, int64_t capacity, int32_t nthreads) {
    if (n < 0 || m < 0 || d <= 0 || (d & 7) || capacity < 0 || isnan(r) || r < 0) return -1;
    if (n >= INT32_MAX || m >= INT32_MAX) return -1;
    int nt = resolve_threads(nthreads);
    int64_t nb = num_blocks(n, nt);
    pairbuf *blk = (pairbuf *)calloc((size_t)nb, sizeof(pairbuf));
    if (!blk) return -1;
    const size_t rb = (size_t)d / 8;
#pragma omp parallel for schedule(dynamic, 1) num_threads(nt)
    for (int64_t b = 0; b < nb; ++b) {
        int64_t i0 = n * b / nb, i1 = n * (b + 1) / nb;
        for (int64_t i = i0; i < i1; ++i)
            for (int64_t j = 0; j < m; ++j)
                if ((double)oracle_hamming_bits(P + (size_t)i * rb, Q + (size_t)j * rb, d) <= r) pb_push(&blk[b], i, j);
    }
    return gather(blk, nb, out_pairs, capacity);
}

/* ------------------------------------------------------------------ LSH-bucketed join
 * Section 4's second algorithm: L repetitions; in each, every point gets a hash that concatenates k
 * base hashes, the points are split into buckets by that hash, and the brute-force join runs inside
 * each bucket; the result is the union over the repetitions.  With a fixed hash family the result is
 * therefore exactly { (i, j) in the brute-force join : the hashes of x_i and y_j agree in at least
 * one repetition } -- which is what this oracle enumerates, with no buckets at all.
 * Base hash, family 0 (bit sampling, the classic monotone LSH for Hamming / +-1 data): h(x) = [x_c > 0] for a
 * sampled coordinate c; the k bits of a repetition sample k distinct coordinates (lsh_rep_coordinates below) from
 * a counter-based generator that the CUDA library implements on its own.
 * Base hash, family 1 (random hyperplanes, the LSH of the angular distance): h(x) = [<a, x> > 0] for a vector a of
 * independent random signs (oracle_lsh_hp_sign below); a projection of exactly zero gives bit 0.
 * When the number of base hashes the analysis asks for is not an integer, the paper builds L_high
 * tables from ceil(k) base hashes and L_low tables from floor(k): here the first L_high repetitions
 * use k bits and the following L_low use k - 1. */
static uint64_t splitmix64_at(uint64_t seed, uint64_t idx) {
    uint64_t z = seed + (idx + 1) * 0x9E3779B97F4A7C15ULL;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

/* The coordinates sampled by the bits of repetition `rep`: bit b takes the first of
 *     splitmix64(seed, 64 rep + b + 4096 a) mod d,   a = 0, 1, 2, ...
 * that no earlier bit of the repetition took -- bit sampling without replacement, so that a repetition of k bits
 * really has 2^k buckets (sampled with replacement, k = 7 of d = 128 coordinates repeat one in 15 % of the
 * repetitions).  From bit d on every coordinate is taken and a = 0 is used as it comes. */
static int lsh_iid_sampling = 0;      /* 1: the k bits of a repetition are k independent samples (a coordinate may repeat) */

/* Chooses between the two bit-sampling rules for the calls that follow: distinct coordinates within a repetition (0, the
 * default) or the paper's plain concatenation of k independent base hashes (1), for which a pair at Hamming distance h
 * collides in a repetition with probability exactly (1 - h/d)^k. */
void oracle_lsh_set_iid_sampling(int32_t on) { lsh_iid_sampling = on != 0; }

static void lsh_rep_coordinates(uint64_t seed, int32_t rep, int32_t bits, int32_t d, int32_t *coord) {
    for (int32_t b = 0; b < bits; ++b) {
        for (uint64_t a = 0;; ++a) {
            int32_t c = (int32_t)(splitmix64_at(seed, (uint64_t)rep * 64u + (uint64_t)b + 4096u * a) % (uint64_t)d);
            int taken = 0;
            for (int32_t e = 0; e < b && b < d && !lsh_iid_sampling; ++e) taken |= coord[e] == c;
            if (!taken) { coord[b] = c; break; }
        }
    }
}

int32_t oracle_lsh_coordinate(uint64_t seed, int32_t rep, int32_t bit, int32_t d) {
    int32_t coord[64];
    if (bit < 0 || bit >= 64) return -1;
    lsh_rep_coordinates(seed, rep, bit + 1, d, coord);
    return coord[bit];
}

/* keys[l * rows + i] = the hash of row i in repetition l (bit b = [x_{c(l,b)} > 0]); k bits in the
 * first L_high repetitions, k - 1 in the next L_low. */
void oracle_lsh_keys_i8(const int8_t *X, int64_t rows, int32_t d, int32_t L_high, int32_t L_low, int32_t k, uint64_t seed,
                        uint32_t *keys) {
    for (int32_t l = 0; l < L_high + L_low; ++l) {
        int32_t coord[64];
        const int32_t bits = l < L_high ? k : k - 1;
        lsh_rep_coordinates(seed, l, bits, d, coord);
        for (int64_t i = 0; i < rows; ++i) {
            uint32_t key = 0;
            for (int32_t b = 0; b < bits; ++b)
                if (X[(size_t)i * d + coord[b]] > 0) key |= 1u << b;
            keys[(size_t)l * rows + i] = key;
        }
    }
}

/* The same keys for bf16 rows: bit b = [x_{c(l,b)} > 0] on the value the 16-bit pattern denotes (+-0 -> 0).  For
 * rows drawn from a rotation-invariant distribution this is the random-hyperplane hash of the angular distance with
 * axis-aligned hyperplanes: two points at angle theta agree on a sampled sign with probability 1 - theta / pi. */
void oracle_lsh_keys_bf16(const uint16_t *X, int64_t rows, int32_t d, int32_t L_high, int32_t L_low, int32_t k, uint64_t seed,
                          uint32_t *keys) {
    for (int32_t l = 0; l < L_high + L_low; ++l) {
        int32_t coord[64];
        const int32_t bits = l < L_high ? k : k - 1;
        lsh_rep_coordinates(seed, l, bits, d, coord);
        for (int64_t i = 0; i < rows; ++i) {
            uint32_t key = 0;
            for (int32_t b = 0; b < bits; ++b)
                if (oracle_bf16_to_f64(X[(size_t)i * d + coord[b]]) > 0.0) key |= 1u << b;
            keys[(size_t)l * rows + i] = key;
        }
    }
}

/* ---- family 1: sign random projections ----
 * Hyperplane of repetition `rep`, bit `bit`: a vector of d independent random signs, coordinate c being +1 when bit 0
 * of splitmix64(seed, 2^60 + (64 rep + bit) 2^20 + c) is set and -1 otherwise (rows of at most 2^20 coordinates).
 * Random-sign vectors have the angular collision law of Gaussian ones in the limit of many coordinates of
 * comparable size: two points at angle theta agree on a bit with probability 1 - theta / pi, whatever the
 * distribution of the data (no rotation invariance needed, unlike the sampled-coordinate sign). */
int32_t oracle_lsh_hp_sign(uint64_t seed, int32_t rep, int32_t bit, int32_t c) {
    const uint64_t idx = (1ULL << 60) + (((uint64_t)rep * 64u + (uint64_t)bit) << 20) + (uint64_t)c;
    return (splitmix64_at(seed, idx) & 1u) ? 1 : -1;
}

/* keys[l * rows + i]: bit b = [ sum_c a_{l,b,c} x_{i,c} > 0 ], the sum an exact integer; k bits in the first L_high
 * repetitions, k - 1 (the same hyperplanes without the last) in the next L_low. */
void oracle_lsh_keys_hp_i8(const int8_t *X, int64_t rows, int32_t d, int32_t L_high, int32_t L_low, int32_t k, uint64_t seed,
                           uint32_t *keys) {
    for (int32_t l = 0; l < L_high + L_low; ++l) {
        const int32_t bits = l < L_high ? k : k - 1;
        for (int64_t i = 0; i < rows; ++i) keys[(size_t)l * rows + i] = 0;
        for (int32_t b = 0; b < bits; ++b) {
            int32_t *a = (int32_t *)malloc(sizeof(int32_t) * (size_t)d);           /* the hyperplane, written out once */
            if (!a) return;
            for (int32_t c = 0; c < d; ++c) a[c] = oracle_lsh_hp_sign(seed, l, b, c);
            for (int64_t i = 0; i < rows; ++i) {
                int64_t proj = 0;
                for (int32_t c = 0; c < d; ++c) proj += (int64_t)a[c] * (int64_t)X[(size_t)i * d + c];
                if (proj > 0) keys[(size_t)l * rows + i] |= 1u << b;
            }
            free(a);
        }
    }
}

/* The same for bf16 rows, projections summed in fp64 with c ascending.  A floating-point sign decides a bit here, and
 * an implementation that accumulates in fp32 may decide a projection close to zero the other way: `unsure` (may be
 * NULL) gets, per repetition and row, the mask of the bits with |projection| <= tol * sum_c |x_c|; a comparison of
 * hash keys leaves those bits free. */
void oracle_lsh_keys_hp_bf16(const uint16_t *X, int64_t rows, int32_t d, int32_t L_high, int32_t L_low, int32_t k, uint64_t seed,
                             double tol, uint32_t *keys, uint32_t *unsure) {
    for (int32_t l = 0; l < L_high + L_low; ++l) {
        const int32_t bits = l < L_high ? k : k - 1;
        for (int64_t i = 0; i < rows; ++i) {
            keys[(size_t)l * rows + i] = 0;
            if (unsure) unsure[(size_t)l * rows + i] = 0;
        }
        for (int32_t b = 0; b < bits; ++b) {
            double *a = (double *)malloc(sizeof(double) * (size_t)d);              /* the hyperplane, written out once */
            if (!a) return;
            for (int32_t c = 0; c < d; ++c) a[c] = (double)oracle_lsh_hp_sign(seed, l, b, c);
            for (int64_t i = 0; i < rows; ++i) {
                double proj = 0.0, mass = 0.0;
                for (int32_t c = 0; c < d; ++c) {
                    const double v = oracle_bf16_to_f64(X[(size_t)i * d + c]);
                    proj += a[c] * v;
                    mass += fabs(v);
                }
                if (proj > 0.0) keys[(size_t)l * rows + i] |= 1u << b;
                if (unsure && fabs(proj) <= tol * mass) unsure[(size_t)l * rows + i] |= 1u << b;
            }
            free(a);
        }
    }
}

int64_t oracle_lsh_join_i8(const int8_t *P, int64_t n, const int8_t *Q, int64_t m, int32_t d, double threshold,
                           int32_t L_high, int32_t L_low, int32_t k, uint64_t seed, int32_t *out_pairs, int64_t capacity,
                           int32_t nthreads) {
    const int32_t L = L_high + L_low;
    if (n < 0 || m < 0 || d <= 0 || capacity < 0 || isnan(threshold) || L_high < 0 || L_low < 0 || L < 1 || L > 64 || k < 0 ||
        k > 20 || (L_low > 0 && k < 1))
        return -1;
    if (n >= INT32_MAX || m >= INT32_MAX) return -1;
    int nt = resolve_threads(nthreads);
    uint32_t *KP = (uint32_t *)malloc(((size_t)L * n + 1) * sizeof(uint32_t));
    uint32_t *KQ = (uint32_t *)malloc(((size_t)L * m + 1) * sizeof(uint32_t));
    int64_t nb = num_blocks(n, nt);
    pairbuf *blk = (pairbuf *)calloc((size_t)nb, sizeof(pairbuf));
    int64_t total = -1;
    if (KP && KQ && blk) {
        oracle_lsh_keys_i8(P, n, d, L_high, L_low, k, seed, KP);
        oracle_lsh_keys_i8(Q, m, d, L_high, L_low, k, seed, KQ);
#pragma omp parallel for schedule(dynamic, 1) num_threads(nt)
        for (int64_t b = 0; b < nb; ++b) {
            int64_t i0 = n * b / nb, i1 = n * (b + 1) / nb;
            for (int64_t i = i0; i < i1; ++i)
                for (int64_t j = 0; j < m; ++j) {
                    int collide = 0;
                    for (int32_t l = 0; l < L && !collide; ++l) collide = KP[(size_t)l * n + i] == KQ[(size_t)l * m + j];
                    if (collide && (double)oracle_ip_i8(P + (size_t)i * d, Q + (size_t)j * d, d) >= threshold) pb_push(&blk[b], i, j);
                }
        }
        total = gather(blk, nb, out_pairs, capacity);
    } else {
        free(blk);
    }
    free(KP);
    free(KQ);
    return total;
}

/* ------------------------------------------------------------------ JL transform
 * Section 3 (the lemma that constructs M and its proof): M = (I_{r_l} (x) A_l) ... (I_{r_1} (x) A_1),
 * applied to a vector level by level: level i cuts its input into r_i consecutive blocks of c_i
 * coordinates and maps every block with the same k_i x c_i matrix A_i.  Sizes as the proof sets them,
 * with zeta = 2 (the value the running-time theorem uses): l = log2(d / k), r_i = 2^(l-i),
 * k_i = i*k for i < l and k_l = k, c_1 = 2k, c_i = 2*k_(i-1).  A_i: independent random signs scaled by
 * 1/sqrt(k_i) (the paper allows any matrix family with the strong JL moment property and names random
 * +-1 entries); sign of entry (a, b) of A_i = bit 0 of splitmix64(seed, i * 2^40 + a * c_i + b):
 * 1 -> +1, 0 -> -1.  Everything in fp64; inputs are bf16 bit patterns, widened exactly. */
int32_t oracle_jl_levels(int32_t d, int32_t k) {
    if (d <= 0 || k <= 0 || d % k != 0) return -1;
    int32_t q = d / k, l = 0;
    while (q > 1 && q % 2 == 0) { q /= 2; ++l; }
    return (q == 1 && l >= 1) ? l : -1;
}

/* (r_i, c_i, k_i) of level i (1-based); returns 0 on success. */
int32_t oracle_jl_shape(int32_t d, int32_t k, int32_t i, int32_t *r, int32_t *c, int32_t *kout) {
    const int32_t l = oracle_jl_levels(d, k);
    if (l < 1 || i < 1 || i > l) return -1;
    *r = 1 << (l - i);
    *kout = i < l ? i * k : k;
    *c = i == 1 ? 2 * k : 2 * (i - 1) * k;
    return 0;
}

int32_t oracle_jl_sign(uint64_t seed, int32_t level, int64_t a, int64_t b, int32_t c_i) {
    return (splitmix64_at(seed, ((uint64_t)level << 40) + (uint64_t)(a * c_i + b)) & 1u) ? 1 : -1;
}

/* out (rows x k, fp64) = M applied to every row of X (rows x d, bf16 bits).  Returns 0, or -1 for bad sizes. */
int32_t oracle_jl_transform_bf16(const uint16_t *X, int64_t rows, int32_t d, int32_t k, uint64_t seed, double *out) {
    const int32_t l = oracle_jl_levels(d, k);
    if (l < 1 || rows < 0) return -1;
    double *cur = (double *)malloc(sizeof(double) * (size_t)d);
    double *nxt = (double *)malloc(sizeof(double) * (size_t)d);
    if (!cur || !nxt) { free(cur); free(nxt); return -1; }
    for (int64_t row = 0; row < rows; ++row) {
        for (int32_t t = 0; t < d; ++t) cur[t] = oracle_bf16_to_f64(X[(size_t)row * d + t]);
        for (int32_t i = 1; i <= l; ++i) {
            int32_t r, c, ki;
            oracle_jl_shape(d, k, i, &r, &c, &ki);
            const double scale = 1.0 / sqrt((double)ki);
            for (int32_t blk = 0; blk < r; ++blk)
                for (int32_t a = 0; a < ki; ++a) {
                    double acc = 0.0;
                    for (int32_t b = 0; b < c; ++b) acc += (double)oracle_jl_sign(seed, i, a, b, c) * cur[(size_t)blk * c + b];
                    nxt[(size_t)blk * ki + a] = acc * scale;
                }
            double *tmp = cur; cur = nxt; nxt = tmp;
        }
        for (int32_t t = 0; t < k; ++t) out[(size_t)row * k + t] = cur[t];
    }
    free(cur);
    free(nxt);
    return 0;
}

int64_t oracle_join_bf16(const uint16_t *P, int64_t n, const uint16_t *Q, int64_t m, int32_t d, int32_t kind,
                         double threshold, int32_t *out_pairs, int64_t capacity, int32_t nthreads) {
    if (n < 0 || m < 0 || d <= 0 || capacity < 0 || kind < KIND_IP || kind > KIND_L2) return -1;
    if (isnan(threshold) || (kind == KIND_L2 && threshold < 0)) return -1;
    if (n >= INT32_MAX || m >= INT32_MAX) return -1;
    int nt = resolve_threads(nthreads);
    double *WP = widen_rows(P, n, d), *WQ = widen_rows(Q, m, d);
    double *NP = WP ? row_sq_norms(WP, n, d) : NULL, *NQ = WQ ? row_sq_norms(WQ, m, d) : NULL;
    int64_t nb = num_blocks(n, nt);
    pairbuf *blk = (pairbuf *)calloc((size_t)nb, sizeof(pairbuf));
    int64_t total = -1;
    if (WP && WQ && NP && NQ && blk) {
#pragma omp parallel for schedule(dynamic, 1) num_threads(nt)
        for (int64_t b = 0; b < nb; ++b) {
            int64_t i0 = n * b / nb, i1 = n * (b + 1) / nb;
            for (int64_t i = i0; i < i1; ++i)
                for (int64_t j = 0; j < m; ++j) {
                    double s = score_f64(WP + (size_t)i * d, WQ + (size_t)j * d, d, kind, NP[i], NQ[j]);
                    if (pass_f64(s, kind, threshold)) pb_push(&blk[b], i, j);
                }
        }
        total = gather(blk, nb, out_pairs, capacity);
    } else {
        free(blk);
    }
    free(WP);
    free(WQ);
    free(NP);
    free(NQ);
    return total;
}
