/*
 * simjoin.h -- C ABI of the B200 (sm_100a) thresholded all-pairs similarity join.
 *
 * The operation is the similarity join of Section 4 of arXiv 2006.12608:
 *   P join_r Q = { (x, y) : x in P, y in Q, D(x, y) <= r }
 * for the ip-distances that section lists, evaluated by the brute-force route
 * it describes: the product F_P * G_Q^T, decomposed into small dense tile
 * products (Theorem 1) that run on the tensor cores.  Rows are identified by
 * their index, so the result is a set of index pairs (i, j), 0-based, i a row
 * of P and j a row of Q.  The n x m score matrix is never materialised: the
 * threshold and the compaction of passing pairs are fused behind each tile
 * product.
 *
 * Conventions
 *   - "device pointer": memory of the context's CUDA device (e.g. the
 *     data_ptr() of a torch tensor).  "host pointer": ordinary host memory.
 *   - Matrices are row-major with the d coordinates of a point contiguous.
 *     Rows must start on 16-byte boundaries: the base pointer is 16-byte
 *     aligned and d * sizeof(element) is a multiple of 16 (pad with zero
 *     columns otherwise: zero columns change no score).
 *   - Nothing the caller passes is freed or retained after a call returns.
 *     P and Q are only read.
 *   - No function throws, prints or exits; every failure is a status code.  (With SIMJOIN_DEBUG=1 in the
 *     environment simjoin_run writes one line per join to stderr: sizes, geometry, variant choice, count.)
 *   - A context is not thread-safe; use one per host thread / stream.
 */
#ifndef SIMJOIN_H_
#define SIMJOIN_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct simjoin_ctx simjoin_ctx; /* opaque; owned by the library */

typedef enum {
    SIMJOIN_I8 = 0,  /* int8 coordinates, exact int32 accumulation              */
    SIMJOIN_BF16 = 1 /* bfloat16 coordinates, fp32 accumulation                 */
} simjoin_dtype;

typedef enum {
    SIMJOIN_IP = 0,  /* keep (i,j) when <x_i, y_j>                  >= threshold */
    SIMJOIN_COS = 1, /* keep (i,j) when <x_i, y_j>/(|x_i| |y_j|)    >= threshold;
                        the cosine with a zero vector counts as 0                */
    SIMJOIN_L2 = 2   /* keep (i,j) when |x_i - y_j| <= threshold (threshold >= 0),
                        evaluated as |x|^2 + |y|^2 - 2<x,y> <= threshold^2; bf16
                        radii too small for that form in fp32 are decided from
                        the rows as sum (x - y)^2 <= threshold^2                 */
} simjoin_kind;

typedef enum {
    SIMJOIN_OK = 0,
    SIMJOIN_ERR_ARG = 1,         /* null / negative / NaN / wrong pointer kind    */
    SIMJOIN_ERR_UNSUPPORTED = 2, /* alignment, d too large, dtype x kind missing  */
    SIMJOIN_ERR_CAPACITY = 3,    /* more passing pairs than `capacity`            */
    SIMJOIN_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed           */
    SIMJOIN_ERR_TIMEOUT = 5,     /* a bounded wait inside the kernel ran out      */
    SIMJOIN_ERR_ARCH = 6         /* the device is not compute capability 10.x     */
} simjoin_status;

/* Limits of this build. */
#define SIMJOIN_MAX_ROWS 2147483647LL /* n, m < 2^31 (pairs are int32)          */
#define SIMJOIN_MAX_ROW_BYTES 8192    /* d * sizeof(element) <= 8192             */

/*
 * Create a context for joins over `dtype` points on CUDA device `device`,
 * enqueueing on `cuda_stream` (a cudaStream_t; NULL = the legacy default
 * stream).  The stream stays owned by the caller and must outlive the context.
 * The context owns its scratch (row norms, per-tile norm bounds, two 64-byte
 * control blocks and a pinned host mirror that the kernel writes its result to,
 * staging buffers of simjoin_run_host, the buffers of the widened entry points),
 * grown on demand with cudaMalloc and released by simjoin_destroy.
 * Errors: ERR_ARG (null ctx, unknown dtype, bad device), ERR_ARCH, ERR_CUDA.
 */
simjoin_status simjoin_create(simjoin_ctx **ctx, simjoin_dtype dtype, int device, void *cuda_stream);

/*
 * The join (Section 4: join definition; brute-force product F_P * G_Q^T).
 *
 *   P, Q        device pointers, n x d and m x d, row-major, read-only.
 *   kind        see simjoin_kind.  Supported: {I8, BF16} x {IP, COS, L2}.
 *   threshold   t (IP, COS) or r (L2).  I8/IP passes when the integer score s
 *               satisfies s >= t over the reals; I8/L2 when the integer squared
 *               distance D satisfies D <= floor(r*r), r*r the double product;
 *               I8/COS when the fp64 quotient <x,y> / sqrt(|x|^2 |y|^2) is >= t
 *               (exact integer sums and product; the conversion to double, the
 *               square root and the quotient each rounded once; 0 for a zero
 *               vector) -- int8 results are exact, with no tolerance band.
 *               BF16 kinds compare fp32 scores; pairs whose exact score lies
 *               within 1e-2*|threshold| of the threshold may fall on either side,
 *               and only those -- at every threshold the call accepts.  (BF16/L2:
 *               the norm expansion's fp32 rounding error, bounded from the largest
 *               norms the pre-pass meets, is compared with 1.9 % of r^2 on the
 *               device; when it is larger the tile test only raises candidates,
 *               lowered by that bound, and each is decided in the difference
 *               form from its two rows.  r = 0 returns exactly the equal rows.
 *               BF16/IP and BF16/COS: where the band is narrower than the fp32
 *               accumulation error of the tile product -- t = 0 above all, where
 *               it is empty -- the tile test likewise only raises candidates and
 *               each is decided from its two rows in fp64, products exact, sums
 *               over k ascending: the exact decision.  Cosine: chosen by the
 *               host, |t| below ~200 error bounds; inner product: chosen on
 *               the device from the largest norms, for which every BF16/IP join
 *               runs the norm pre-pass.  A BF16 cosine threshold beyond +-2
 *               decides like +-2.)
 *   out_pairs   device pointer to capacity x 2 int32, written as (i, j) rows.
 *               May be NULL when capacity == 0 (count-only mode).
 *   count       HOST pointer; receives the total number of passing pairs, even
 *               when that exceeds `capacity`.
 *
 * Exactly min(*count, capacity) rows of out_pairs are written, each passing
 * pair at most once, in unspecified order.  When *count > capacity the written
 * subset is arbitrary but valid and the call returns ERR_CAPACITY.
 * The call enqueues on the context's stream and synchronises that stream
 * once, before it returns (no host round trip in between: which variant of
 * the kernel runs -- 16- or 32-bit int8 epilogue, BF16/L2 small-radius form --
 * is decided on the device).  n == 0 or m == 0 gives OK with *count = 0.
 *
 * Errors, all detected before any launch: ERR_ARG (null ctx/P/Q/count, n or m
 * negative or >= 2^31, d <= 0, NaN threshold, L2 with threshold < 0, a host
 * pointer where a device pointer is required, out_pairs NULL with capacity > 0);
 * ERR_UNSUPPORTED (misaligned base pointer, d*sizeof(element) not a multiple
 * of 16 or above SIMJOIN_MAX_ROW_BYTES).  After launch: ERR_CUDA,
 * ERR_TIMEOUT (a wait in the kernel gave up; the context stays usable),
 * ERR_CAPACITY.
 */
simjoin_status simjoin_run(simjoin_ctx *ctx, const void *P, int64_t n, const void *Q, int64_t m,
                           int32_t d, simjoin_kind kind, double threshold, int32_t *out_pairs,
                           uint64_t capacity, uint64_t *count);

/*
 * Same join with HOST buffers: P, Q and out_pairs are host pointers.  The call
 * copies P and Q to device staging owned by the context, runs the join, and
 * copies min(*count, capacity) pairs back; all on the context's stream,
 * synchronised before return.  Pinned host memory makes the copies faster but
 * is not required.  A Q above 64 MiB is uploaded in slices of about 32 MiB (one of 32 to 64 MiB in four slices) on a second stream and every
 * slice is joined as soon as it has landed, so that (with pinned memory) the copies of later slices hide
 * behind the joins of earlier ones; the result is the union of the slices' results.  With room for 64 MiB of
 * pairs or more (capacity >= 2^23) Q is cut into eight slices whatever its size, and the pairs of a slice are
 * copied to out_pairs_host while the next slice is joined (dense results: the download hides behind the joins).
 * Errors as simjoin_run (device pointers are rejected here).
 */
simjoin_status simjoin_run_host(simjoin_ctx *ctx, const void *P_host, int64_t n, const void *Q_host,
                                int64_t m, int32_t d, simjoin_kind kind, double threshold,
                                int32_t *out_pairs_host, uint64_t capacity, uint64_t *count);

#define SIMJOIN_LSH_MAX_REPS 64
#define SIMJOIN_LSH_MAX_BITS 12

/*
 * LSH-bucketed join (Section 4, the algorithm after the brute-force one): repetitions;
 * in each, every point is hashed with a concatenation of base hashes from an LSH family, the points
 * are split into buckets by that hash, and the brute-force tile join runs inside each bucket; the
 * result is the union over the repetitions.  For a fractional number of base hashes the paper mixes
 * tables built from ceil(k) and floor(k) base hashes: here L repetitions use k bits and L_low more
 * use k - 1 (the same samples without the last).  The output is therefore exactly
 *     { (i, j) of simjoin_run(kind, threshold)  with  key_l(x_i) == key_l(y_j) for some repetition l },
 * a subset of simjoin_run's (precision 1; the recall is set by L, k and the data; bf16: the same threshold band
 * as simjoin_run).
 *
 *   family        the LSH family (the paper takes it as a black box: "an (r, cr, p1, p2)-sensitive monotone LSH").
 *     SIMJOIN_LSH_BITS         bit sampling: h(x) = [x_c > 0] for a sampled coordinate c -- the standard family for
 *                 Hamming distance, i.e. for +-1 rows such as simjoin_run_hamming builds; for bf16 rows the
 *                 sign of the sampled coordinate, i.e. the random-hyperplane hash of the angular distance
 *                 with axis-aligned hyperplanes (two rows of a rotation-invariant distribution at angle
 *                 theta agree with probability 1 - theta/pi).  The k bits of a repetition sample k DISTINCT
 *                 coordinates (without replacement, so that the repetition has 2^k buckets): bit b of
 *                 repetition l takes the first of splitmix64(seed, 64*l + b + 4096*a) mod d, a = 0, 1, ...,
 *                 that no earlier bit of the repetition took (from bit d on, a = 0 as it comes), where
 *                 splitmix64(seed, i): z = seed + (i+1)*0x9E3779B97F4A7C15; z = (z ^ z>>30)*0xBF58476D1CE4E5B9;
 *                 z = (z ^ z>>27)*0x94D049BB133111EB; z ^ z>>31  (all modulo 2^64).
 *     SIMJOIN_LSH_BITS_IID     bit sampling as the paper states it, "a concatenation of k independent base hashes": bit b of
 *                 repetition l samples splitmix64(seed, 64*l + b) mod d whether or not an earlier bit took that coordinate
 *                 (a repetition with a repeated coordinate has fewer, larger buckets).  A pair at Hamming distance h then
 *                 collides in a repetition with probability exactly (1 - h/d)^k, the p1^k of the paper's analysis.
 *     SIMJOIN_LSH_HYPERPLANES  random hyperplanes (sign random projections), the LSH of the angular distance for data of
 *                 any shape: h(x) = [<a, x> > 0], a projection of exactly zero giving 0; a is a vector of random signs,
 *                 coordinate c of the hyperplane of repetition l, bit b being +1 when bit 0 of
 *                 splitmix64(seed, 2^60 + (64 l + b) 2^20 + c) is set and -1 otherwise.  Two points at angle theta agree
 *                 on a bit with probability 1 - theta/pi.  The projections of all points onto all hyperplanes are one
 *                 dense product, computed by the tile kernel on the tensor cores (16 hyperplane rows per repetition,
 *                 a sign-collecting epilogue that writes the key records).  int8: the projections are exact integers
 *                 and the keys exact; bf16: fp32 accumulation, so a projection within about (d + 64) 2^-23 sum |x_c| of
 *                 zero may hash to either side (such a point may land in either of two buckets of that repetition).
 *   P, Q, n, m, d, kind, threshold, out_pairs, capacity, count   as simjoin_run (every dtype and kind it accepts).
 *   L, L_low      repetitions with k and with k - 1 bits (the first k - 1 samples / hyperplanes of their k); both >= 0,
 *                 1 <= L + L_low <= SIMJOIN_LSH_MAX_REPS, L_low > 0 needs k >= 1 (ERR_ARG otherwise; also for an
 *                 unknown family).
 *   k             key bits, 0..SIMJOIN_LSH_MAX_BITS (ERR_ARG if negative, ERR_UNSUPPORTED above);
 *                 k = 0 puts everything in one bucket and returns the brute-force result.
 *
 * Every pair is reported once, whatever the number of
 * repetitions it collides in; the order is unspecified.  The context keeps regrouped copies of P and Q
 * and two copies of a record of 16-bit keys per row as scratch:
 * (n+m) * (row bytes + 4 + 32*ceil((L+L_low)/8)) bytes (+ 4 per row for the norm kinds).  Hashing, regrouping, the work list and the bucketed
 * join all run on the device with no host round trip between repetitions.
 * simjoin_last_kernel_ms then reports (hashing, all repetitions).
 */
typedef enum { SIMJOIN_LSH_BITS = 0, SIMJOIN_LSH_HYPERPLANES = 1, SIMJOIN_LSH_BITS_IID = 2 } simjoin_lsh_family;
simjoin_status simjoin_run_lsh(simjoin_ctx *ctx, const void *P, int64_t n, const void *Q, int64_t m, int32_t d,
                               simjoin_kind kind, double threshold, simjoin_lsh_family family, int32_t L, int32_t L_low,
                               int32_t k, uint64_t seed, int32_t *out_pairs, uint64_t capacity, uint64_t *count);

/*
 * LSH-bucketed Hamming join on bit-packed points: simjoin_run_hamming's operand transform followed by
 * simjoin_run_lsh -- bit sampling is the LSH family of the Hamming distance, so bit b of the key of repetition l is
 * simply the coordinate of the point that simjoin_run_lsh samples for that bit.  The output is exactly
 *     { (i, j) : Hamming(x_i, y_j) <= r  and  key_l(x_i) == key_l(y_j) for some repetition l }.
 * Arguments as simjoin_run_hamming (P_bits, Q_bits, n, m, d, r) and simjoin_run_lsh (L, L_low, k, seed); errors
 * as those two.  I8 contexts only.
 */
simjoin_status simjoin_run_hamming_lsh(simjoin_ctx *ctx, const void *P_bits, int64_t n, const void *Q_bits, int64_t m,
                                       int32_t d, double r, int32_t L, int32_t L_low, int32_t k, uint64_t seed,
                                       int32_t *out_pairs, uint64_t capacity, uint64_t *count);

/*
 * JL transform (Section 3: the lemma that builds M = (I_{r_l} (x) A_l) ... (I_{r_1} (x) A_1) and computes M x
 * as l small dense products): out = X M^T for all n rows at once, reducing d coordinates to k, as a
 * pre-reduction before an (approximate) join on the k-dimensional rows.
 *
 *   X     device pointer, n x d bf16, row-major, 16-byte aligned.          out   device pointer, n x k bf16.
 *   d, k  d / k must be a power of two >= 2 (zeta = 2, the value of the paper's running-time theorem; l =
 *         log2(d / k) levels; ERR_ARG otherwise); k a multiple of 8 and 2*(l-1)*k*2 bytes <= SIMJOIN_MAX_ROW_BYTES
 *         (ERR_UNSUPPORTED otherwise).  The paper's k = ceil(C eps^-2 log 1/delta) has an unspecified constant:
 *         k is the caller's choice.
 *   Level i (1..l) cuts every point into r_i = 2^(l-i) blocks of c_i coordinates (c_1 = 2k, c_i = 2(i-1)k) and
 *   maps each block with the same k_i x c_i matrix A_i (k_i = i*k, k_l = k) of independent random signs scaled
 *   by 1/sqrt(k_i); the sign of entry (a, b) is bit 0 of splitmix64(seed, i * 2^40 + a * c_i + b) (1 -> +1),
 *   splitmix64 as in simjoin_run_lsh.  Each level is one launch of the tile kernel with A_i resident in shared
 *   memory and the blocks streamed by TMA; products are exact in fp32 up to accumulation order, and each level's
 *   output is rounded to bf16 (the next level's operand type).
 *
 * BF16 contexts only (ERR_UNSUPPORTED otherwise).  Scratch owned by the context: two buffers of n * max_i(r_i k_i)
 * bf16 values and one level matrix.  Synchronises the stream before returning.  simjoin_last_kernel_ms then
 * reports (0, all levels).
 */
simjoin_status simjoin_jl_transform(simjoin_ctx *ctx, const void *X, int64_t n, int32_t d, int32_t k, uint64_t seed,
                                    void *out);

/*
 * Hamming join on bit-packed points (Section 4: Hamming is the first ip-distance listed, with the
 * embedding f(x) = (x_k, 1-x_k)_k, g(y) = (1-y_k, y_k)_k).  keep (i, j) when Hamming(x_i, y_j) <= r.
 *
 *   P_bits, Q_bits  device pointers, n and m rows of d/8 bytes; coordinate k of a row is bit k%8
 *                   (least significant first) of byte k/8.  d must be a multiple of 128 (16-byte rows),
 *                   base pointers 16-byte aligned.  I8 contexts only (ERR_UNSUPPORTED otherwise).
 *   r               >= 0; a real r acts as floor(r).  ERR_ARG for NaN or negative r.
 *
 * The library applies the operand transform x -> 2x-1 on the device (bits to +-1 int8 rows in staging
 * owned by the context: d' = d instead of the paper's 2d, because <x+-, y+-> = d - 2*Hamming) and runs
 * the int8 inner-product join with threshold d - 2*floor(r).  Result, count, capacity and error
 * semantics are those of simjoin_run; the pair set is exact.
 */
simjoin_status simjoin_run_hamming(simjoin_ctx *ctx, const void *P_bits, int64_t n, const void *Q_bits, int64_t m,
                                   int32_t d, double r, int32_t *out_pairs, uint64_t capacity, uint64_t *count);

/*
 * Candidate filter (Section 4's join definition applied to a list of pairs instead of all of P x Q): keeps the
 * listed pairs (i, j) for which (row i of P, row j of Q) passes `kind` at `threshold`, and drops the others.
 *
 *   P, Q, n, m, d, kind, threshold   as simjoin_run.
 *   pairs       device pointer to count_in x 2 int32, 8-byte aligned: indices as the joins of this context emit them
 *               (row offsets of simjoin_set_offsets included).  Compacted in place; the order of the kept pairs is
 *               unspecified.  An index outside [0, n) x [0, m) makes the call return ERR_ARG (the list is then
 *               unspecified, nothing outside it is touched).
 *   count_out   HOST pointer; number of pairs kept.
 *
 * Arithmetic: I8 exact (the decisions simjoin_run takes); BF16 in fp32 -- inner product and cosine as sums over
 * the row, the Euclidean distance in the difference form sum (x - y)^2 <= r^2 (no cancellation of large norms);
 * a pair whose exact score lies within 1e-2*|threshold| of the threshold may fall on either side.  An inner product or
 * cosine whose fp32 value lies within the sums' rounding error of the threshold is decided again in fp64 (exact
 * products, k ascending), so thresholds at or next to zero, whose band is empty, are decided exactly too.
 * A group of lanes per pair (sized to the row), two rows read per pair.  Synchronises the stream.  Scratch: count_in x 8 bytes.
 */
simjoin_status simjoin_filter_pairs(simjoin_ctx *ctx, const void *P, int64_t n, const void *Q, int64_t m, int32_t d,
                                    simjoin_kind kind, double threshold, int32_t *pairs, uint64_t count_in,
                                    uint64_t *count_out);

/*
 * Euclidean join behind a JL pre-reduction (Section 3's transform used as the paper introduces it: reduce the
 * dimension, then search): both point sets are reduced from d to k coordinates with the same matrix M
 * (simjoin_jl_transform, same seed), the reduced points are joined with the radius widened to r * (1 + slack)
 * (the reduced rows of Q ordered by norm first, which keeps the join's per-block bounds tight),
 * and the candidates are decided on the original rows (simjoin_filter_pairs, radius r).  The result is a subset
 * of the exact join { (i, j) : |x_i - y_j| <= r } (band rule of simjoin_filter_pairs): a true pair is missed only
 * when M stretches its distance by more than 1 + slack.  With random-sign levels the relative spread of |M z| / |z|
 * is about 1 / sqrt(2k) per level; slack = 0.3 at k = 64 loses well under 1 % of the pairs.
 *
 *   P, Q        device pointers, n x d and m x d bf16.  d, k, seed: as simjoin_jl_transform.  slack >= 0.
 *   out_pairs, capacity, count: as simjoin_run; the capacity must hold the CANDIDATES (when it does not, the call
 *               returns ERR_CAPACITY with *count = the number of candidates and out_pairs unspecified).
 *
 * BF16 contexts only.  Scratch: the two reduced sets ((n + m) x k bf16) plus that of the calls above.
 * simjoin_last_kernel_ms then reports (both transforms, reduced join + filter).
 */
simjoin_status simjoin_run_jl_l2(simjoin_ctx *ctx, const void *P, int64_t n, const void *Q, int64_t m, int32_t d, double r,
                                 int32_t k, uint64_t seed, double slack, int32_t *out_pairs, uint64_t capacity,
                                 uint64_t *count);

/*
 * Row squared norms, the pre-pass behind the |x|^2 and |y|^2 terms of the
 * squared-L2 and cosine ip-distances (Section 4).  X: device pointer, rows x d.
 * out: device pointer to `rows` values -- int32 (exact) for I8 contexts, fp32
 * for BF16 contexts.  Synchronises the stream before returning.
 * Errors: ERR_ARG, ERR_UNSUPPORTED (alignment / row bytes as above), ERR_CUDA.
 */
simjoin_status simjoin_row_norms(simjoin_ctx *ctx, const void *X, int64_t rows, int32_t d, void *out);

/*
 * Offsets added to every emitted pair: (i + row_offset_p, j + row_offset_q).
 * Lets a caller that shards P (or Q) by row blocks over several GPUs or calls
 * obtain global indices directly (Theorem 1's block decomposition: the union
 * of the joins of the blocks is the join).  Both default to 0.  The sums must
 * stay below 2^31: ERR_ARG otherwise (checked again in simjoin_run).
 */
simjoin_status simjoin_set_offsets(simjoin_ctx *ctx, int64_t row_offset_p, int64_t row_offset_q);

/*
 * Tuning knobs of a context; none of them changes a result.
 *
 *   SIMJOIN_OPT_SELECT_MIN_OPS   int8 joins of at least this many operations (2 n m d) run the max|x| pre-pass and let
 *                                the device choose the 16-bit packed epilogue when every score provably fits 16 bits;
 *                                smaller joins take the 32-bit epilogue unasked, which saves two steps of launch latency
 *                                (default 2e11; 0 = always ask).  value >= 0.
 *   SIMJOIN_OPT_KERNEL_TIMING    1 (default): simjoin_run records CUDA events around its pre-pass and its join kernel
 *                                for simjoin_last_kernel_ms; 0: it records none (three stream operations less per call,
 *                                which shows on joins of a few microseconds) and simjoin_last_kernel_ms reports ERR_ARG.
 *   SIMJOIN_OPT_DENSE_EPILOGUE   which epilogue layout bf16 joins over rows of one or two whole 128-byte chunks run
 *                                (d = 64 or 128): 0 = always 8 epilogue warps of 128 columns (best when pairs are rare:
 *                                the work is row maxima); 1 = always 16 warps of 64 columns (best when most 32 x 128
 *                                blocks of scores hold a pair: the work is element tests, bound by dependent-issue
 *                                latency, which twice the warps hide; measured 77.5 -> 70.8 ms on 2.7e8 pairs out of
 *                                524 288^2, +2 % on a join with 1000 pairs out of 65 536^2); 2 (default) = by the
 *                                previous simjoin_run of the context: 16 warps after a join with at least one pair per
 *                                two such blocks; a context that has run no join yet counts the pairs of a sample first
 *                                (its first 256 rows of P against 128 rows of Q per SM) when the join has at least
 *                                1e12 operations.  A join in the 16-warp layout whose rows are at most 240 bytes long
 *                                (under 2: after a join with at least one pair per block) runs as the sign test of one
 *                                inner product on transformed operands -- Section 4's ip-distance embeddings with the
 *                                threshold folded in: 8 coordinates appended to context-owned copies of both point sets
 *                                ((n + m) x 128 or 256 bytes of scratch) so that <x', y'> >= 0 exactly when the pair
 *                                passes.  Euclidean: (r^2 - |x|^2)/2 and -|y|^2/2 in three bf16 pieces each against ones
 *                                (70.8 -> 42.3 ms on the same join); inner product: -t in three pieces against ones;
 *                                cosine: the six largest piece products of (-t |x|) |y| and two flags for zero vectors
 *                                (18.3 -> 10.4 ms on 6.7e7 pairs out of 262 144^2, d = 64).  Euclidean radii too small for
 *                                the fp32 norm expansion still take the row-deciding form on the points themselves.
 *                                Other joins ignore the option.
 * Errors: ERR_ARG (null ctx, unknown option, NaN or out-of-range value).
 */
typedef enum { SIMJOIN_OPT_SELECT_MIN_OPS = 0, SIMJOIN_OPT_KERNEL_TIMING = 1, SIMJOIN_OPT_DENSE_EPILOGUE = 2 } simjoin_option;
simjoin_status simjoin_set_option(simjoin_ctx *ctx, simjoin_option option, double value);

/*
 * Device time of the kernels of the last successful simjoin_run /
 * simjoin_run_host on this context, in milliseconds, measured with CUDA events
 * on the context's stream: the norm pre-pass (0 when the kind needs none) and
 * the join kernel.  Either pointer may be NULL.  ERR_ARG if nothing has run.
 */
simjoin_status simjoin_last_kernel_ms(simjoin_ctx *ctx, float *prepass_ms, float *join_ms);

/*
 * Self-test of the kernel's failure path.  Every wait inside the join kernel is bounded: when one
 * expires the kernel raises a status word, drains and returns, and the call reports ERR_TIMEOUT
 * with the context still usable.  This entry point launches a one-warp kernel that waits, with a
 * ~1 ms budget, on a barrier nothing ever completes, and reads the status back the same way
 * simjoin_run does.  Returns SIMJOIN_ERR_TIMEOUT when the path works (the expected result),
 * SIMJOIN_ERR_CUDA otherwise.  It faults nothing and leaves the context usable.
 */
simjoin_status simjoin_selftest_wait_timeout(simjoin_ctx *ctx);

/*
 * Allocation-free join.  (The paper has no counterpart: this entry point exists for the
 * sake of callers, not of the method.)
 *
 * Some callers must not trigger a device allocation while they run: a serving loop whose
 * memory is handed out once by a pool and whose latency budget cannot absorb the implicit
 * device synchronisation of cudaMalloc / cudaFree, a plugin that runs under a host
 * framework owning all device memory, code on a path where an out-of-memory failure is not
 * an option.  simjoin_create / simjoin_run grow scratch with cudaMalloc; this call does not.
 * It calls no cudaMalloc, cudaFree, cudaMallocHost, event or stream creation, nor any other
 * allocating routine: the scratch of the pre-passes and of the join kernel (row norms,
 * per-tile norm bounds, the counter / status / selection block) lives in a fixed array inside
 * the library's device image, about 0.5 MiB that every GPU loading the library holds until the
 * process exits.  There is no context: device, stream and dtype are arguments.  From the
 * choice of the tile geometry on it is simjoin_run's own code path -- the same pre-passes,
 * the same kernel instantiations for every row length, the same device-side choice of
 * variant -- only the working memory differs.
 *
 * Same semantics, supported kinds and error codes as simjoin_run, with these differences:
 *   - n and m must not exceed SIMJOIN_NOALLOC_MAX_ROWS; larger inputs are rejected with
 *     SIMJOIN_ERR_UNSUPPORTED before anything is launched (use simjoin_run instead).
 *   - emitted indices carry no offsets; no kernel timings are recorded.
 *   - the first call on each device looks up the device address of the scratch array and
 *     sets kernel attributes; make that first call before any stream capture begins, and
 *     not concurrently with another first call on the same device.
 *   - all calls on a device share the one scratch array, which keeps the previous call's
 *     contents (this call clears the words that must start at zero).  Two calls whose
 *     kernels overlap on the GPU -- different streams, or different host threads -- race
 *     on it and give wrong results: serialise them.
 * P, Q, out_pairs are device pointers, count a host pointer, exactly as in simjoin_run;
 * the call synchronises `cuda_stream` before it returns.
 */
#define SIMJOIN_NOALLOC_MAX_ROWS 65536
simjoin_status simjoin_run_noalloc(int device, void *cuda_stream, simjoin_dtype dtype, const void *P, int64_t n,
                                   const void *Q, int64_t m, int32_t d, simjoin_kind kind, double threshold,
                                   int32_t *out_pairs, uint64_t capacity, uint64_t *count);

/* Release the context and its scratch.  NULL is accepted. */
simjoin_status simjoin_destroy(simjoin_ctx *ctx);

/* Static, human-readable name of a status code. */
const char *simjoin_strerror(simjoin_status status);

#ifdef __cplusplus
}
#endif
#endif /* SIMJOIN_H_ */
