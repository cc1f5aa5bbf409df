// Candidate filter: given a list of index pairs (i, j), keep those whose rows pass the join's predicate
// (Section 4's definition, applied to listed pairs instead of all of P x Q).  It closes the approximate pipeline
// "reduce with the JL transform of Section 3, join the short rows with some slack, decide the candidates on the
// original rows": whatever distortion the reduction adds, only true pairs leave.
// A group of G lanes per pair (G = the power of two covering the row's 16-byte words, at most 32: a warp takes
// 32 / G pairs at a time, so that short rows keep all lanes loading): the lanes stride over the words of the two rows,
// three running sums are reduced with shuffles inside the group, its first lane decides and appends the pair to the
// output list (one atomic per kept pair; order unspecified).  HBM/L2-bound: 2 rows per candidate.  A listed index outside the point sets raises a status bit and is skipped.
#pragma once
#include <cstdint>

#include "lsh_kernel.cuh"   // block_scan4 and the counting-sort kernels

namespace sj {

constexpr int FILTER_THREADS = 256;

// int8 rows: exact integer sums.  IP: s >= ceil(t) (thr_i);  L2: sum (x-y)^2 <= floor(r^2) (thr_i), taken as
// |x|^2 + |y|^2 - 2s in integers;  COS: the fp64 sequence of the join's exact test (thr_d).
// bf16 rows: fp32 sums.  IP: s >= t;  COS: s >= t |x| |y|, a zero vector scoring 0;  L2: the difference form
// sum (x-y)^2 <= r^2, which does not cancel like the norm expansion of the tile epilogue.  An inner product or cosine
// whose fp32 value lies within the sums' rounding error ((d + 32) 2^-23 |x| |y|) of the threshold is decided again in
// fp64 (exact products, k ascending, the fp64 threshold): whatever the threshold -- zero included, where the tolerance
// band 1e-2 |t| is empty -- the decision is the one exact arithmetic takes.
template <int DT, int KIND>
__global__ void __launch_bounds__(FILTER_THREADS)
filter_pairs_kernel(const uint4 *__restrict__ P, long long n, const uint4 *__restrict__ Q, long long m, int g,
                    const int2 *__restrict__ in, unsigned long long count_in, int ioff, int joff, int thr_i, float thr_f,
                    double thr_d, int2 *__restrict__ out, unsigned long long *__restrict__ counter,
                    unsigned int *__restrict__ status, int G) {
    const int wlane = threadIdx.x & 31;
    const int lane = wlane & (G - 1), sub = wlane / G, ppw = 32 / G;      // lane within the pair's group; pairs per warp
    const unsigned long long warp = ((unsigned long long)blockIdx.x * FILTER_THREADS + threadIdx.x) >> 5;
    const unsigned long long nwarps = ((unsigned long long)gridDim.x * FILTER_THREADS) >> 5;
    for (unsigned long long k0 = warp * ppw; k0 < count_in; k0 += nwarps * ppw) {      // warp-uniform trip count
        const unsigned long long k = k0 + sub;
        int2 pr = make_int2(0, 0);
        bool live = k < count_in;
        if (live) {
            pr = in[k];
            const long long li = (long long)pr.x - ioff, lj = (long long)pr.y - joff;
            if (li < 0 || li >= n || lj < 0 || lj >= m) {  // not a pair of these point sets: flag it, touch nothing
                if (lane == 0) atomicOr(status, 0x20000000u);
                live = false;
            }
        }
        const uint4 *x = P + (live ? (long long)pr.x - ioff : 0) * g, *y = Q + (live ? (long long)pr.y - joff : 0) * g;
        const int gl = live ? g : 0;                       // a dead group loads nothing but keeps shuffling
        bool pass = false;
        if constexpr (DT == DT_I8) {
            int s = 0, nx = 0, ny = 0;
            for (int c = lane; c < gl; c += G) {
                const uint4 a = __ldg(x + c), b = __ldg(y + c);
                const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    s = __dp4a((int)aw[t], (int)bw[t], s);
                    nx = __dp4a((int)aw[t], (int)aw[t], nx);
                    ny = __dp4a((int)bw[t], (int)bw[t], ny);
                }
            }
            for (int off = G >> 1; off > 0; off >>= 1) {
                s += __shfl_xor_sync(0xffffffffu, s, off);
                nx += __shfl_xor_sync(0xffffffffu, nx, off);
                ny += __shfl_xor_sync(0xffffffffu, ny, off);
            }
            if constexpr (KIND == KIND_IP) pass = s >= thr_i;
            if constexpr (KIND == KIND_L2) pass = (long long)nx + ny - 2LL * s <= (long long)thr_i;
            if constexpr (KIND == KIND_COS) {
                if (nx == 0 || ny == 0) pass = 0.0 >= thr_d;
                else pass = __ddiv_rn((double)s, __dsqrt_rn(__ll2double_rn((long long)nx * (long long)ny))) >= thr_d;
            }
        } else {
            float s = 0.f, nx = 0.f, ny = 0.f;       // L2: s accumulates the squared differences
            for (int c = lane; c < gl; c += G) {
                const uint4 a = __ldg(x + c), b = __ldg(y + c);
                const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const float x0 = __uint_as_float(aw[t] << 16), x1 = __uint_as_float(aw[t] & 0xffff0000u);
                    const float y0 = __uint_as_float(bw[t] << 16), y1 = __uint_as_float(bw[t] & 0xffff0000u);
                    if constexpr (KIND == KIND_L2) {
                        const float e0 = x0 - y0, e1 = x1 - y1;
                        s = fmaf(e0, e0, s);
                        s = fmaf(e1, e1, s);
                    } else {
                        s = fmaf(x0, y0, s);
                        s = fmaf(x1, y1, s);
                    }
                    if constexpr (KIND != KIND_L2) {
                        nx = fmaf(x0, x0, nx);
                        nx = fmaf(x1, x1, nx);
                        ny = fmaf(y0, y0, ny);
                        ny = fmaf(y1, y1, ny);
                    }
                }
            }
            for (int off = G >> 1; off > 0; off >>= 1) {
                s += __shfl_xor_sync(0xffffffffu, s, off);
                if constexpr (KIND != KIND_L2) {
                    nx += __shfl_xor_sync(0xffffffffu, nx, off);
                    ny += __shfl_xor_sync(0xffffffffu, ny, off);
                }
            }
            if constexpr (KIND == KIND_L2) pass = s <= thr_f;
            if constexpr (KIND != KIND_L2) {
                const float nn = sqrtf(nx) * sqrtf(ny);
                const float b = KIND == KIND_IP ? thr_f : thr_f * nn;
                pass = s >= b;
                const float margin = (float)(g * 8 + 32) * 0x1p-23f * nn;
                // (a comparison that is false for a NaN or infinite margin also takes the slow path)
                if (live && lane == 0 && !(fabsf(s - b) > margin)) {
                    double s2 = 0.0, nx2 = 0.0, ny2 = 0.0;
                    for (int c = 0; c < g; ++c) {
                        const uint4 a = __ldg(x + c), bb = __ldg(y + c);
                        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {bb.x, bb.y, bb.z, bb.w};
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            const double x0 = (double)__uint_as_float(aw[t] << 16), x1 = (double)__uint_as_float(aw[t] & 0xffff0000u);
                            const double y0 = (double)__uint_as_float(bw[t] << 16), y1 = (double)__uint_as_float(bw[t] & 0xffff0000u);
                            s2 = __dadd_rn(s2, __dmul_rn(x0, y0));
                            s2 = __dadd_rn(s2, __dmul_rn(x1, y1));
                            nx2 = __dadd_rn(nx2, __dmul_rn(x0, x0));
                            nx2 = __dadd_rn(nx2, __dmul_rn(x1, x1));
                            ny2 = __dadd_rn(ny2, __dmul_rn(y0, y0));
                            ny2 = __dadd_rn(ny2, __dmul_rn(y1, y1));
                        }
                    }
                    if constexpr (KIND == KIND_IP) pass = s2 >= thr_d;
                    else pass = (nx2 == 0.0 || ny2 == 0.0) ? 0.0 >= thr_d : __ddiv_rn(s2, __dmul_rn(__dsqrt_rn(nx2), __dsqrt_rn(ny2))) >= thr_d;
                }
            }
        }
        if (live && lane == 0 && pass) out[atomicAdd(counter, 1ULL)] = pr;
    }
}

// ---- ordering rows by norm (the reduced join of simjoin_run_jl_l2) ----
// The tile epilogue prunes with a bound built from the smallest |y|^2 of a 256-row block of Q.  Reduced rows have
// norms that spread by +-1/sqrt(k/2) around the original ones, which loosens that bound; with the rows of Q ordered
// by norm every block is nearly constant.  A counting sort on a 12-bit quantisation of the norm is enough.

// range[0] = min, range[1] = max of the (non-negative) norms, as float bits (whose integer order is the floats').
__global__ void __launch_bounds__(256) norm_range_kernel(const float *__restrict__ ny, long long m, unsigned int *range) {
    unsigned int mn = 0x7f7f7f7fu, mx = 0u;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < m; i += (long long)gridDim.x * blockDim.x) {
        const unsigned int b = __float_as_uint(ny[i]);
        mn = min(mn, b);
        mx = max(mx, b);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        mn = min(mn, __shfl_xor_sync(0xffffffffu, mn, off));
        mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    }
    if ((threadIdx.x & 31) == 0) {
        atomicMin(range, mn);
        atomicMax(range + 1, mx);
    }
}

// key[i] in [0, nb): the position of ny[i] between the smallest and the largest norm.
__global__ void __launch_bounds__(256) norm_keys_kernel(const float *__restrict__ ny, long long m, const unsigned int *__restrict__ range,
                                                        int nb, uint16_t *__restrict__ keys) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= m) return;
    const float lo = __uint_as_float(range[0]), hi = __uint_as_float(range[1]);
    const float span = hi - lo;
    int key = span > 0.f ? (int)((ny[i] - lo) / span * (float)nb) : 0;
    keys[i] = (uint16_t)min(max(key, 0), nb - 1);
}

// cursor[b] = number of rows with a key below b (one block; nb <= 4096).
__global__ void __launch_bounds__(1024) hist_offsets_kernel(const unsigned int *__restrict__ hist, int nb, unsigned int *__restrict__ cursor) {
    __shared__ unsigned int s_warp[33];
    unsigned int v[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) v[t] = threadIdx.x * 4 + t < nb ? hist[threadIdx.x * 4 + t] : 0u;
    block_scan4(v, s_warp);
#pragma unroll
    for (int t = 0; t < 4; ++t)
        if (threadIdx.x * 4 + t < nb) cursor[threadIdx.x * 4 + t] = v[t];
}

// pairs[t].y: position in the ordered copy (+ joff) -> original row (+ joff).
__global__ void __launch_bounds__(256) remap_second_index_kernel(int2 *__restrict__ pairs, unsigned long long count,
                                                                 const int *__restrict__ perm, int joff) {
    const unsigned long long t = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t < count) pairs[t].y = perm[pairs[t].y - joff] + joff;
}

}  // namespace sj
