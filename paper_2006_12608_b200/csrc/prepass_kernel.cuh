// Row-norm pre-pass: |x|^2 per row (the |x|^2, |y|^2 terms of Section 4's squared-L2
// ip-distance and the 1/|x| scaling of its cosine form), plus, per 256-row tile, the
// minimum and maximum of the stored values, which the join kernel turns into a per-tile
// bound that lets it skip whole blocks of the score tile.  Memory-bound: every input
// byte is read once with 16-byte loads.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>

namespace sj {

constexpr int NORM_TILE_ROWS = 256;
constexpr int NORM_THREADS = 256;

template <bool kInt8>
struct NormAcc;
template <>
struct NormAcc<true> {
    using type = int;
    static __device__ __forceinline__ int add16(int acc, const uint4 &q) {
        acc = __dp4a((int)q.x, (int)q.x, acc);
        acc = __dp4a((int)q.y, (int)q.y, acc);
        acc = __dp4a((int)q.z, (int)q.z, acc);
        acc = __dp4a((int)q.w, (int)q.w, acc);
        return acc;
    }
};
template <>
struct NormAcc<false> {
    using type = float;
    static __device__ __forceinline__ float add16(float acc, const uint4 &q) {
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const float lo = __uint_as_float(w[t] << 16), hi = __uint_as_float(w[t] & 0xffff0000u);
            acc = fmaf(lo, lo, acc);
            acc = fmaf(hi, hi, acc);
        }
        return acc;
    }
};

// One warp, 32 consecutive rows of G 16-byte chunks each (G a power of two <= 32): G lanes share a
// row; the row sums land in out[0..31].
template <bool kInt8, int G>
__device__ __forceinline__ void warp_rows_pow2(const uint4 *__restrict__ X, long long rows, long long row0, int lane,
                                               typename NormAcc<kInt8>::type *out) {
    using T = typename NormAcc<kInt8>::type;
    constexpr int RPP = 32 / G;                 // rows per pass
    constexpr int BATCH = G < 8 ? G : 8;        // passes whose loads are in flight together
    const int sub = lane / G, chunk = lane - sub * G;
#pragma unroll
    for (int p0 = 0; p0 < G; p0 += BATCH) {
        uint4 q[BATCH];
#pragma unroll
        for (int b = 0; b < BATCH; ++b) {
            const long long r = row0 + (p0 + b) * RPP + sub;
            q[b] = r < rows ? __ldg(X + r * G + chunk) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int b = 0; b < BATCH; ++b) {
            T acc = NormAcc<kInt8>::add16(T(0), q[b]);
#pragma unroll
            for (int off = G >> 1; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
            if (chunk == 0) out[(p0 + b) * RPP + sub] = acc;
        }
    }
}

// X: rows x (g * 16 bytes).  norms[r] = sum of squares of row r; with sqrt_out its square root in fp32 (int8
// rows too: the bits of the float in the int32 array, whose order is the floats' order); sqrt_out == 2 stores
// +inf for a zero row.  tile_minmax[b] = (min, max) of norms over the valid rows of tile b (may be null).
// all_max (may be null): the largest stored value of the whole launch, folded in with one atomicMax per block on
// its bit pattern (stored values are non-negative, so the patterns order like the values).
template <bool kInt8>
__global__ void __launch_bounds__(NORM_THREADS)
row_norms_kernel(const uint4 *__restrict__ X, long long rows, int g, int sqrt_out,
                 typename NormAcc<kInt8>::type *__restrict__ norms,
                 typename NormAcc<kInt8>::type *__restrict__ tile_minmax, unsigned int *__restrict__ all_max) {
    using T = typename NormAcc<kInt8>::type;
    __shared__ T s_val[NORM_TILE_ROWS];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long row0 = (long long)blockIdx.x * NORM_TILE_ROWS + warp * 32;   // this warp's 32 rows
    const bool pow2 = g <= 32 && (g & (g - 1)) == 0;
    if (pow2) {
        // g lanes share a row: 32/g rows per pass, g passes; all loads of a warp are contiguous.
        // Loads are issued in batches of up to 8 before anything is reduced (bytes in flight).
        switch (g) {
            case 1: warp_rows_pow2<kInt8, 1>(X, rows, row0, lane, s_val + warp * 32); break;
            case 2: warp_rows_pow2<kInt8, 2>(X, rows, row0, lane, s_val + warp * 32); break;
            case 4: warp_rows_pow2<kInt8, 4>(X, rows, row0, lane, s_val + warp * 32); break;
            case 8: warp_rows_pow2<kInt8, 8>(X, rows, row0, lane, s_val + warp * 32); break;
            case 16: warp_rows_pow2<kInt8, 16>(X, rows, row0, lane, s_val + warp * 32); break;
            default: warp_rows_pow2<kInt8, 32>(X, rows, row0, lane, s_val + warp * 32); break;
        }
    } else {
        for (int rl = 0; rl < 32; ++rl) {
            const long long r = row0 + rl;
            T acc = 0;
            if (r < rows)
                for (int c = lane; c < g; c += 32) acc = NormAcc<kInt8>::add16(acc, __ldg(X + r * g + c));
            for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
            if (lane == 0) s_val[warp * 32 + rl] = acc;
        }
    }
    __syncthreads();
    const long long r = (long long)blockIdx.x * NORM_TILE_ROWS + threadIdx.x;
    T v = s_val[threadIdx.x];
    if constexpr (!kInt8) {
        if (sqrt_out) v = (v == 0.f && sqrt_out == 2) ? __int_as_float(0x7f800000) : sqrtf(v);
    }
    if constexpr (kInt8) {
        if (sqrt_out) v = __float_as_int(v == 0 && sqrt_out == 2 ? __int_as_float(0x7f800000) : sqrtf((float)v));
    }
    const bool valid = r < rows;
    if (valid) norms[r] = v;
    if (tile_minmax == nullptr && all_max == nullptr) return;
    // block min / max over valid rows (row 0 of a launched tile is always valid)
    __syncthreads();
    s_val[threadIdx.x] = v;
    __syncthreads();
    const T first = s_val[0];
    T mn = valid ? v : first, mx = mn;
    for (int off = 16; off > 0; off >>= 1) {
        const T a = __shfl_xor_sync(0xffffffffu, mn, off), b = __shfl_xor_sync(0xffffffffu, mx, off);
        mn = a < mn ? a : mn;
        mx = b > mx ? b : mx;
    }
    __shared__ T s_mn[NORM_THREADS / 32], s_mx[NORM_THREADS / 32];
    if (lane == 0) { s_mn[warp] = mn; s_mx[warp] = mx; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < NORM_THREADS / 32; ++w) {
            mn = s_mn[w] < mn ? s_mn[w] : mn;
            mx = s_mx[w] > mx ? s_mx[w] : mx;
        }
        if (tile_minmax != nullptr) {
            tile_minmax[2 * (long long)blockIdx.x] = mn;
            tile_minmax[2 * (long long)blockIdx.x + 1] = mx;
        }
        if (all_max != nullptr) {
            unsigned int bits;
            if constexpr (kInt8) bits = (unsigned int)mx;
            else bits = __float_as_uint(mx);
            atomicMax(all_max, bits);
        }
    }
}

// max |x| over two int8 buffers of nP16 and nQ16 16-byte words, folded into out[0] (P) and out[1] (Q) with
// atomicMax; the first half of the grid reads P, the second Q.  The join kernel proves from these two words that
// d * max|P| * max|Q| fits in 16 bits before it takes the packed epilogue.
__global__ void __launch_bounds__(256) maxabs_i8_kernel(const uint4 *__restrict__ P, long long nP16, const uint4 *__restrict__ Q,
                                                        long long nQ16, unsigned int *out) {
    const unsigned int half = gridDim.x >> 1;
    const bool second = blockIdx.x >= half;
    const uint4 *X = second ? Q : P;
    const long long n16 = second ? nQ16 : nP16;
    const unsigned int blk = second ? blockIdx.x - half : blockIdx.x, nblk = second ? gridDim.x - half : half;
    unsigned int m = 0;   // four unsigned byte maxima
    for (long long i = (long long)blk * blockDim.x + threadIdx.x; i < n16; i += (long long)nblk * blockDim.x) {
        const uint4 q = __ldg(X + i);
        m = __vmaxu4(m, __vmaxu4(__vmaxu4(__vabs4(q.x), __vabs4(q.y)), __vmaxu4(__vabs4(q.z), __vabs4(q.w))));
    }
    unsigned int v = max(max(m & 0xffu, (m >> 8) & 0xffu), max((m >> 16) & 0xffu, m >> 24));
    v = __reduce_max_sync(0xffffffffu, v);
    if ((threadIdx.x & 31) == 0 && v > 0) atomicMax(out + (second ? 1 : 0), v);
}

// Operand transform for the Hamming ip-distance (Section 4): bit-packed {0,1} coordinates -> +-1 int8
// rows, so that <x, y> = d - 2 * Hamming(x, y) and the int8 inner-product join applies with d' = d.
// One thread expands 16 bits (coordinate k = bit k%8 of byte k/8) into 16 bytes: 1 -> +1, 0 -> -1.
__global__ void __launch_bounds__(256) unpack_bits_pm1_kernel(const uint16_t *__restrict__ bits, long long nhalf,
                                                              uint4 *__restrict__ out) {
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= nhalf) return;
    const uint32_t h = bits[t];
    uint32_t w[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const uint32_t nib = (h >> (4 * q)) & 0xfu;
        const uint32_t ones = (nib * 0x00204081u) & 0x01010101u;        // bit i of the nibble -> byte i
        w[q] = ones | ((ones ^ 0x01010101u) * 0xffu);                   // 0x01 where set, 0xff (-1) where clear
    }
    out[t] = make_uint4(w[0], w[1], w[2], w[3]);
}

// An fp32 value as three bf16 pieces of 8 significant bits each (truncation keeps every remainder exact): h = p1 + p2 + p3.
__device__ __forceinline__ void split3_bf16(float h, uint32_t &b1, uint32_t &b2, uint32_t &b3) {
    const float p1 = __uint_as_float(__float_as_uint(h) & 0xffff0000u);
    const float r1 = h - p1;
    const float p2 = __uint_as_float(__float_as_uint(r1) & 0xffff0000u);
    const float p3 = r1 - p2;                                            // at most 8 significant bits are left
    b1 = __float_as_uint(p1) >> 16;
    b2 = __float_as_uint(p2) >> 16;
    b3 = __float_as_uint(p3) >> 16;
}

// Operand transforms that turn a thresholded ip-distance of Section 4 into the sign of one inner product: 8 coordinates are
// appended to every bf16 row so that <x', y'> >= 0 exactly when the pair passes.  The tile epilogue then needs no per-row or
// per-column term and its element test is the score's sign bit.
//   EMBED_L2  (Section 4 lists f(x) = (x_k^2, 1, -2 x_k)_k, g(y) = (1, y_k^2, y_k)_k; the same inner product with the
//             squares summed up front):
//                 P side (x, a1, a2, a3, 1, 1, 1, 0, 0)      Q side (y, 1, 1, 1, b1, b2, b3, 0, 0)
//             a1 + a2 + a3 = (r^2 - |x|^2) / 2 and b1 + b2 + b3 = -|y|^2 / 2 exactly, so <x', y'> = (r^2 - |x - y|^2) / 2.
//             norms: |x|^2 in fp32 as the norm pre-pass left it; shift: r^2 on the P side, 0 on the Q side.
//   EMBED_IP  <x, y> >= t:   P side (x, c1, c2, c3, 0, ...) with c1 + c2 + c3 = -t (shift = t), Q side (y, 1, 1, 1, 0, ...).
//   EMBED_COS <x, y> >= t |x| |y| (f = g = x / |x| of Section 4, cleared of the division): with u = -t |x| and v = |y| split
//             into pieces, the product u v is the sum of the nine piece products, of which the six largest are kept (the
//             rest is below 2^-23 of it):
//                 P side (x, u1, u1, u1, u2, u2, u3, zx, 1)    Q side (y, v1, v2, v3, v1, v2, v1, 1, zy)
//             norms: |x| in fp32; a zero vector is stored as +inf when t > 0 (it passes nothing): its pieces are zero and its
//             flag zx (zy) is -1, which makes every score it takes part in negative.  shift = t on the P side.
// Output rows are gout >= g + 1 16-byte words long (whole 128-byte chunks, so that every row of a TMA box is one aligned
// line; measured 65.1 -> 62 ms on the dense 524 288^2 Euclidean join against rows of exactly g + 1 words), zero past the
// appended coordinates.  One thread per output word.
constexpr int EMBED_L2 = 0, EMBED_IP = 1, EMBED_COS = 2;
__global__ void __launch_bounds__(256) embed_rows_kernel(const uint4 *__restrict__ X, const float *__restrict__ norms, long long rows,
                                                         int g, int gout, int mode, int q_side, float shift, uint4 *__restrict__ out) {
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= rows * gout) return;
    const long long r = t / gout;
    const int c = (int)(t - r * gout);
    if (c != g) {
        out[t] = c < g ? __ldg(X + r * g + c) : make_uint4(0u, 0u, 0u, 0u);
        return;
    }
    const uint32_t one = 0x3F80u, minus_one = 0xBF80u;
    uint32_t b1, b2, b3;
    // eight bf16 values, low half of a word first
    if (mode == EMBED_L2) {
        split3_bf16(0.5f * (shift - norms[r]), b1, b2, b3);
        if (q_side) out[t] = make_uint4(one | (one << 16), one | (b1 << 16), b2 | (b3 << 16), 0u);
        else out[t] = make_uint4(b1 | (b2 << 16), b3 | (one << 16), one | (one << 16), 0u);
    } else if (mode == EMBED_IP) {
        if (q_side) out[t] = make_uint4(one | (one << 16), one, 0u, 0u);
        else {
            split3_bf16(-shift, b1, b2, b3);
            out[t] = make_uint4(b1 | (b2 << 16), b3, 0u, 0u);
        }
    } else {
        const float nr = norms[r];
        const bool none = nr == __int_as_float(0x7f800000);        // a zero vector under t > 0
        split3_bf16(none ? 0.f : (q_side ? nr : -shift * nr), b1, b2, b3);
        const uint32_t z = none ? minus_one : 0u;
        if (q_side) out[t] = make_uint4(b1 | (b2 << 16), b3 | (b1 << 16), b2 | (b1 << 16), one | (z << 16));
        else out[t] = make_uint4(b1 | (b1 << 16), b1 | (b2 << 16), b2 | (b3 << 16), z | (one << 16));
    }
}

}  // namespace sj
