// Bucketing kernels of the LSH join (Section 4, second algorithm): hash every point L times with a
// concatenation of k base hashes, and for each repetition regroup the rows of P and Q so that every
// bucket is one contiguous row range, then list the (P row block, Q bucket) units the join kernel sweeps.
//
// Base hash, first family: bit sampling, h(x) = [x_c > 0] for a sampled coordinate c -- the classic monotone family
// for Hamming distance / +-1 data, and for bf16 rows the sign of the sampled coordinate (the random-hyperplane
// hash of the angular distance with axis-aligned hyperplanes; a bf16 value is positive exactly when its bit
// pattern, read as int16, is).  The k bits of a repetition sample k distinct coordinates, drawn from a counter-based
// generator (lsh_coordinates_kernel), so nothing random is stored.
// Second family: random hyperplanes, h(x) = [<a, x> > 0] with a a vector of random signs from the same generator
// (lsh_hyperplanes_kernel); the projections of all points onto all hyperplanes are one dense product, which the
// tile kernel computes with a sign-collecting epilogue (KIND_SIGN).
#pragma once
#include <cstdint>

namespace sj {

constexpr int LSH_MAX_BITS = 12;                    // buckets per repetition <= 4096 (shared-memory histograms)
constexpr int LSH_MAX_BUCKETS = 1 << LSH_MAX_BITS;
constexpr int LSH_MAX_REPS = 64;
constexpr int LSH_SORT_THREADS = 256;
constexpr int LSH_SORT_ITEMS = 8;                   // rows per thread in the scatter kernel

__host__ __device__ inline uint64_t lsh_splitmix64(uint64_t seed, uint64_t idx) {
    uint64_t z = seed + (idx + 1) * 0x9E3779B97F4A7C15ULL;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

// s_coord[l * k + b] = the coordinate bit b of repetition l samples: the first of
//     splitmix64(seed, 64 l + b + 4096 a) mod d,   a = 0, 1, 2, ...
// that no earlier bit of the repetition took (bit sampling without replacement: k bits give 2^k buckets; from bit d
// on, when every coordinate is taken, a = 0 is used as it comes).  One thread per repetition, one block, once per
// call: the key kernels read the table from global memory.
// `distinct` == 0: the k bits are k independent samples (a = 0 always; a coordinate may repeat within a repetition).
__global__ void __launch_bounds__(64) lsh_coordinates_kernel(unsigned long long seed, int L, int k, int d, int distinct, int *__restrict__ coords) {
    for (int l = threadIdx.x; l < L; l += blockDim.x) {
        int *coord = coords + l * k;
        for (int b = 0; b < k; ++b) {
            for (uint64_t a = 0;; ++a) {
                const int c = (int)(lsh_splitmix64(seed, (uint64_t)l * 64u + (uint64_t)b + 4096u * a) % (uint64_t)d);
                bool taken = false;
                for (int e = 0; e < b && b < d && distinct; ++e) taken = taken || coord[e] == c;
                if (!taken) { coord[b] = c; break; }
            }
        }
    }
}
// The hyperplanes of the second family as a matrix for the tile kernel: 16 rows per repetition, row 16 l + b the
// hyperplane of repetition l, bit b -- coordinate c is +1 when bit 0 of splitmix64(seed, 2^60 + (64 l + b) 2^20 + c) is
// set and -1 otherwise -- and zero rows for the bits a repetition does not use (b >= k, or k - 1 in the last L_low
// repetitions) and for the padding repetitions up to `reps_padded`.  T: int8_t, or uint16_t holding bf16 bit patterns.
template <typename T>
__global__ void __launch_bounds__(256) lsh_hyperplanes_kernel(unsigned long long seed, int L_high, int L_low, int k, int d,
                                                              int reps_padded, T *__restrict__ planes) {
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= (long long)reps_padded * 16 * d) return;
    const int c = (int)(t % d), row = (int)(t / d), l = row >> 4, b = row & 15;
    const int bits = l < L_high ? k : (l < L_high + L_low ? k - 1 : 0);
    T val = 0;
    if (b < bits) {
        const bool plus = lsh_splitmix64(seed, (1ULL << 60) + (((uint64_t)l * 64u + (uint64_t)b) << 20) + (uint64_t)c) & 1u;
        if constexpr (sizeof(T) == 1) val = plus ? (T)1 : (T)-1;
        else val = plus ? (T)0x3F80 : (T)0xBF80;            // +-1.0 in bf16
    }
    planes[t] = val;
}

__device__ __forceinline__ void lsh_load_coordinates(const int *__restrict__ coords, int L, int k, int *s_coord) {
    for (int t = threadIdx.x; t < L * k; t += blockDim.x) s_coord[t] = coords[t];
}

// rec[i * stride + l] = key of row i in repetition l (one record of `stride` 16-bit keys per row, so that
// all keys of a row sit in one or two cache lines): k bits in the first L_high repetitions, k - 1 (the
// same samples without the last) in the following L_low -- the paper's mix of tables for a fractional
// number of base hashes.  One thread per row; the sampled coordinates are computed once per block.
template <typename T>   // int8_t, or int16_t for bf16 bit patterns
__global__ void __launch_bounds__(256) lsh_keys_kernel(const T *__restrict__ X, long long rows, int d, int L_high, int L_low,
                                                       int k, const int *__restrict__ coords, uint16_t *__restrict__ rec, int stride) {
    __shared__ int s_coord[LSH_MAX_REPS * LSH_MAX_BITS];
    const int L = L_high + L_low;
    lsh_load_coordinates(coords, L, k, s_coord);
    __syncthreads();
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows) return;
    const T *x = X + i * d;
    for (int l = 0; l < stride; ++l) {
        uint32_t key = 0;
        const int bits = l < L_high ? k : (l < L ? k - 1 : 0);      // padding entries stay 0
        for (int b = 0; b < bits; ++b) key |= (x[s_coord[l * k + b]] > 0 ? 1u : 0u) << b;
        rec[i * stride + l] = (uint16_t)key;
    }
}

// The same keys for short rows (at most LSH_KEYS_STAGED_MAX_D bytes): a block first copies its 64 rows into shared
// memory with coalesced 16-byte loads (row pitch: row bytes + 4, an odd number of words, so the gathers of
// different rows fall into different banks), then four threads per row split the repetitions.  The per-thread
// gather of the kernel above touches 32 different cache lines with every load instruction.
constexpr int LSH_KEYS_STAGED_MAX_D = 512;
constexpr int LSH_KEYS_STAGED_ROWS = 64;
template <typename T>
__global__ void __launch_bounds__(256) lsh_keys_staged_kernel(const T *__restrict__ X, long long rows, int d, int L_high, int L_low,
                                                              int k, const int *__restrict__ coords, uint16_t *__restrict__ rec, int stride) {
    __shared__ int s_coord[LSH_MAX_REPS * LSH_MAX_BITS];
    extern __shared__ uint32_t s_rows[];                       // LSH_KEYS_STAGED_ROWS x (row bytes / 4 + 1) words
    const int L = L_high + L_low;
    lsh_load_coordinates(coords, L, k, s_coord);
    const long long row0 = (long long)blockIdx.x * LSH_KEYS_STAGED_ROWS;
    const int row_bytes = d * (int)sizeof(T);
    const int g = row_bytes / 16, pitch = row_bytes / 4 + 1;
    const uint4 *src = reinterpret_cast<const uint4 *>(X + row0 * d);
    const long long avail = (rows - row0 < LSH_KEYS_STAGED_ROWS ? rows - row0 : LSH_KEYS_STAGED_ROWS) * g;
    for (int t = threadIdx.x; t < LSH_KEYS_STAGED_ROWS * g; t += blockDim.x) {
        if (t >= avail) break;
        const uint4 q = __ldg(src + t);
        const int r = t / g, c = t - r * g;
        uint32_t *dst = s_rows + r * pitch + c * 4;
        dst[0] = q.x; dst[1] = q.y; dst[2] = q.z; dst[3] = q.w;
    }
    __syncthreads();
    const int r = threadIdx.x >> 2, part = threadIdx.x & 3;
    const long long i = row0 + r;
    if (i >= rows) return;
    const T *x = reinterpret_cast<const T *>(s_rows + r * pitch);
    for (int l = part; l < stride; l += 4) {
        uint32_t key = 0;
        const int bits = l < L_high ? k : (l < L ? k - 1 : 0);      // padding entries stay 0
        for (int b = 0; b < bits; ++b) key |= (x[s_coord[l * k + b]] > 0 ? 1u : 0u) << b;
        rec[i * stride + l] = (uint16_t)key;
    }
}

// hist[key] += number of rows with that key (block-private histogram in shared memory first).
// keys: the key of row i is keys[i * stride] (one column of the key records).
__global__ void __launch_bounds__(LSH_SORT_THREADS) lsh_hist_kernel(const uint16_t *__restrict__ keys, int stride, long long rows,
                                                                    int nb, unsigned int *__restrict__ hist) {
    __shared__ unsigned int s_cnt[LSH_MAX_BUCKETS];
    for (int b = threadIdx.x; b < nb; b += blockDim.x) s_cnt[b] = 0;
    __syncthreads();
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < rows; i += (long long)gridDim.x * blockDim.x)
        atomicAdd(&s_cnt[keys[i * stride]], 1u);
    __syncthreads();
    for (int b = threadIdx.x; b < nb; b += blockDim.x)
        if (s_cnt[b]) atomicAdd(&hist[b], s_cnt[b]);
}

// Exclusive scan of up to LSH_MAX_BUCKETS values by one 1024-thread block (4 per thread); returns the total.
__device__ __forceinline__ unsigned int block_scan4(unsigned int (&v)[4], unsigned int *s_warp) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned int mine = v[0] + v[1] + v[2] + v[3];
    unsigned int incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned int t = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += t;
    }
    __syncthreads();                         // s_warp may still be read from a previous scan
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const unsigned int w = s_warp[lane];
        unsigned int wi = w;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned int t = __shfl_up_sync(0xffffffffu, wi, off);
            if (lane >= off) wi += t;
        }
        s_warp[lane] = wi - w;               // exclusive prefix of the warp totals
        if (lane == 31) s_warp[32] = wi;     // grand total
    }
    __syncthreads();
    unsigned int run = s_warp[warp] + incl - mine;
#pragma unroll
    for (int t = 0; t < 4; ++t) {
        const unsigned int x = v[t];
        v[t] = run;
        run += x;
    }
    return s_warp[32];
}

// One block: bucket offsets of P and Q (exclusive scans of the histograms; also copied to the scatter
// cursors) and the work list -- for every bucket that holds points of both sets, one unit per rows_per_unit-row
// block of its P rows, each against all of the bucket's Q rows.  Units of a bucket are adjacent.
__global__ void __launch_bounds__(1024) lsh_offsets_units_kernel(const unsigned int *__restrict__ hist_p,
                                                                 const unsigned int *__restrict__ hist_q, int nb,
                                                                 unsigned int *__restrict__ cursor_p,
                                                                 unsigned int *__restrict__ cursor_q, int4 *__restrict__ units,
                                                                 unsigned int *__restrict__ nunits, int rows_per_unit) {
    __shared__ unsigned int s_warp[33];
    unsigned int pc[4], qc[4], po[4], qo[4], ub[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
        const int b = threadIdx.x * 4 + t;
        pc[t] = b < nb ? hist_p[b] : 0u;
        qc[t] = b < nb ? hist_q[b] : 0u;
        po[t] = pc[t];
        qo[t] = qc[t];
        ub[t] = (pc[t] && qc[t]) ? (pc[t] + rows_per_unit - 1) / rows_per_unit : 0u;
    }
    block_scan4(po, s_warp);
    block_scan4(qo, s_warp);
    const unsigned int total = block_scan4(ub, s_warp);
#pragma unroll
    for (int t = 0; t < 4; ++t) {
        const int b = threadIdx.x * 4 + t;
        if (b >= nb) continue;
        cursor_p[b] = po[t];
        cursor_q[b] = qo[t];
        if (pc[t] && qc[t]) {
            const unsigned int nblk = (pc[t] + rows_per_unit - 1) / rows_per_unit;
            for (unsigned int j = 0; j < nblk; ++j) {
                const unsigned int r0 = j * rows_per_unit;
                const unsigned int rr = pc[t] - r0 < (unsigned)rows_per_unit ? pc[t] - r0 : (unsigned)rows_per_unit;
                units[ub[t] + j] = make_int4((int)(po[t] + r0), (int)rr, (int)qo[t], (int)qc[t]);
            }
        }
    }
    if (threadIdx.x == 0) *nunits = total;
}

// perm[position] = row, positions grouped by key: each block ranks its rows inside shared-memory
// counters, reserves one range per key with a single global atomic, and writes its rows there.
__global__ void __launch_bounds__(LSH_SORT_THREADS) lsh_scatter_kernel(const uint16_t *__restrict__ keys, int stride, long long rows,
                                                                       int nb, unsigned int *__restrict__ cursor,
                                                                       int *__restrict__ perm) {
    __shared__ unsigned int s_cnt[LSH_MAX_BUCKETS];
    for (int b = threadIdx.x; b < nb; b += blockDim.x) s_cnt[b] = 0;
    __syncthreads();
    const long long base = (long long)blockIdx.x * (LSH_SORT_THREADS * LSH_SORT_ITEMS);
    uint32_t key[LSH_SORT_ITEMS];
    unsigned int rank[LSH_SORT_ITEMS];
#pragma unroll
    for (int t = 0; t < LSH_SORT_ITEMS; ++t) {
        const long long i = base + t * LSH_SORT_THREADS + threadIdx.x;
        key[t] = i < rows ? keys[i * stride] : 0u;
        rank[t] = i < rows ? atomicAdd(&s_cnt[key[t]], 1u) : 0u;
    }
    __syncthreads();
    for (int b = threadIdx.x; b < nb; b += blockDim.x) {
        const unsigned int c = s_cnt[b];
        if (c) s_cnt[b] = atomicAdd(&cursor[b], c);
    }
    __syncthreads();
#pragma unroll
    for (int t = 0; t < LSH_SORT_ITEMS; ++t) {
        const long long i = base + t * LSH_SORT_THREADS + threadIdx.x;
        if (i < rows) perm[s_cnt[key[t]] + rank[t]] = (int)i;
    }
}

// out row `pos` = X row perm[pos]; rows are g 16-byte words.
__global__ void __launch_bounds__(256) lsh_gather_rows_kernel(const uint4 *__restrict__ X, const int *__restrict__ perm,
                                                              long long rows, int g, uint4 *__restrict__ out) {
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= rows * g) return;
    const long long pos = t / g;
    const int c = (int)(t - pos * g);
    out[t] = __ldg(X + (long long)__ldg(perm + pos) * g + c);
}

}  // namespace sj
