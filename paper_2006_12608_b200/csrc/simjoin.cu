// Host side of the C ABI declared in include/simjoin.h: argument checks, scratch
// management, TMA descriptors, launches of the pre-pass and the fused join kernel.
#include "../../include/simjoin.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "join_kernel.cuh"
#include "filter_kernel.cuh"
#include "jl_kernel.cuh"
#include "lsh_kernel.cuh"
#include "prepass_kernel.cuh"

static_assert(sj::QSTAT_ROWS == sj::NORM_TILE_ROWS, "the join kernel indexes the per-tile bounds by 256-row blocks");

namespace {

using namespace sj;

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct DevBuf {
    void *ptr = nullptr;
    size_t bytes = 0;
};

// Joins of fewer operations (2 n m d) than this run the 32-bit int8 epilogue without asking whether the 16-bit one
// applies: the max|x| pre-pass and the second launch cost two more steps in the stream's dependent chain (about 13 us
// measured on B200), which the packed epilogue's ~15 % only wins back on joins of ~90 us and more.
constexpr double DEFAULT_SELECT_MIN_OPS = 2.0e11;
// Pairs per 32 x 128 block of scores from which a join counts as dense (its next run takes 16 epilogue warps).
constexpr double DENSE_MIN_PAIRS_PER_BLOCK = 0.5;
// ... and from which a Euclidean join in that layout also runs on transformed operands.  Measured on 262 144^2 mixtures, d = 64,
// 16 against 8 warps: cosine 0.87 / 0.91 / 0.93 / 1.00 of the time at 8 / 2 / 0.5 / 0.125 pairs per block; Euclidean with the
// transform 0.72 / 0.84 / 1.04 / 1.27.
constexpr double EMBED_MIN_PAIRS_PER_BLOCK = 1.0;
// Joins of at least this many operations (2 n m d) sample their output density when the context has no history: below
// it the sample's launch and synchronisation (tens of microseconds) are not worth what the better layout saves.
constexpr double DENSITY_SAMPLE_MIN_OPS = 1e12;
constexpr int MAX_HOST_SLICES = 66;     // simjoin_run_host: a Q of more slices than this goes up in one piece

// Device-side working memory of one join call, and the host words its result lands in.  simjoin_run takes it from the
// context's buffers (grown on demand); the allocation-free entry point points it at a fixed array.
struct JoinScratch {
    void *nx, *ny, *qstat;        // row terms of P (n entries) and Q (whole tiles), (min, max) of ny per 256 rows of Q
    unsigned long long *d_ctrl;   // 64 bytes: [0] pair counter, [1] status word, [2] max|P|, max|Q| (two 32-bit words, int8),
                                  // [3] bit patterns of max|x|^2, max|y|^2 (two 32-bit words, bf16 Euclidean),
                                  // [4] low word: ticket of finished CTAs
    unsigned long long *h_ctrl;   // host copy of words [0] and [1]
    bool h_ctrl_mapped;           // h_ctrl is pinned memory the device can write: the kernel stores the result there
};

}  // namespace

struct simjoin_ctx {
    simjoin_dtype dtype;
    int device;
    cudaStream_t stream;
    int num_sms;
    int max_smem_optin;
    EncodeTiledFn encode;
    DevBuf nx, ny, qstat;               // row terms and per-tile bounds
    DevBuf stage_p, stage_q, stage_out; // device staging of simjoin_run_host
    unsigned long long *d_ctrl;         // two 64-byte control blocks (layout: JoinScratch::d_ctrl)
    unsigned long long *h_ctrl;         // pinned mirror
    int ctrl_clean;                     // the block that the last simjoin_run's kernel left zeroed for the next one, or -1
    double select_min_ops;              // SIMJOIN_OPT_SELECT_MIN_OPS
    bool kernel_timing;                 // SIMJOIN_OPT_KERNEL_TIMING
    cudaEvent_t ev[4];
    bool have_timing;
    float prepass_ms, join_ms;
    long long ioff, joff;
    bool attr_set[2][4][2][3][2];
    bool attr_set_long[2][3][2][2];
    bool attr_set_wideq;
    bool attr_set_dense[3][2][3];
    bool attr_set_embed[3][5];
    int dense_mode;                     // SIMJOIN_OPT_DENSE_EPILOGUE: 0 never, 1 always (where instantiated), 2 by the last join's density
    double last_density;                // pairs per 32 x 128 block of scores in the last successful simjoin_run (-1: none yet)
    cudaStream_t copy_stream;           // simjoin_run_host: uploads of Q slices overlap the joins of earlier slices
    cudaEvent_t copy_ev[MAX_HOST_SLICES + 1];   // one per slice, plus one that orders the copy stream behind earlier work
    DevBuf jl_a, jl_buf[2];             // JL transform: level matrix, ping-pong level outputs
    DevBuf jl_p, jl_q;                  // simjoin_run_jl_l2: the reduced point sets
    DevBuf filter_out;                  // simjoin_filter_pairs: the kept pairs before they replace the list
    // LSH join scratch: hash keys, regrouping permutations, regrouped copies of P and Q, histograms + work list
    DevBuf lsh_keys_p, lsh_keys_q, lsh_perm_p, lsh_perm_q, lsh_sorted_p, lsh_sorted_q, lsh_misc;
    DevBuf lsh_planes;                  // hyperplane family: 16 rows per repetition
    DevBuf emb_p, emb_q;                // dense Euclidean joins: the point sets with the squared-L2 embedding coordinates appended
    bool attr_set_sign[2];
};

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        ok = cudaGetDevice(&prev) == cudaSuccess && cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

// The library prints nothing unless the environment holds SIMJOIN_DEBUG=1: then one line per join on stderr.
bool debug_log() {
    static const bool on = [] {
        const char *v = std::getenv("SIMJOIN_DEBUG");
        return v && v[0] == '1';
    }();
    return on;
}

bool grow(DevBuf &b, size_t bytes) {
    if (bytes <= b.bytes) return true;
    if (b.ptr) cudaFree(b.ptr);
    b.ptr = nullptr;
    b.bytes = 0;
    if (cudaMalloc(&b.ptr, bytes) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    b.bytes = bytes;
    return true;
}

void release(DevBuf &b) {
    if (b.ptr) cudaFree(b.ptr);
    b.ptr = nullptr;
    b.bytes = 0;
}

size_t elem_size(simjoin_dtype t) { return t == SIMJOIN_I8 ? 1 : 2; }

// 1 = device memory of `device`, 0 = host / unregistered / other device.
int is_device_ptr(const void *p, int device) {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, p) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    if (a.type == cudaMemoryTypeDevice || a.type == cudaMemoryTypeManaged) return a.device == device;
    return 0;
}

simjoin_status check_matrix_args(const simjoin_ctx *ctx, const void *X, int64_t rows, int32_t d) {
    if (!X || rows < 0 || rows >= SIMJOIN_MAX_ROWS || d <= 0) return SIMJOIN_ERR_ARG;
    const size_t row_bytes = (size_t)d * elem_size(ctx->dtype);
    if (row_bytes % 16 != 0 || row_bytes > SIMJOIN_MAX_ROW_BYTES) return SIMJOIN_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(X) & 15u) != 0) return SIMJOIN_ERR_UNSUPPORTED;
    return SIMJOIN_OK;
}

simjoin_status check_join_args(const simjoin_ctx *ctx, const void *P, int64_t n, const void *Q, int64_t m, int32_t d,
                               simjoin_kind kind, double threshold, const int32_t *out_pairs, uint64_t capacity,
                               const uint64_t *count) {
    if (!ctx || !count) return SIMJOIN_ERR_ARG;
    if (kind != SIMJOIN_IP && kind != SIMJOIN_COS && kind != SIMJOIN_L2) return SIMJOIN_ERR_ARG;
    if (std::isnan(threshold) || (kind == SIMJOIN_L2 && threshold < 0)) return SIMJOIN_ERR_ARG;
    if (!out_pairs && capacity > 0) return SIMJOIN_ERR_ARG;
    simjoin_status st = check_matrix_args(ctx, P, n, d);
    if (st == SIMJOIN_OK || st == SIMJOIN_ERR_UNSUPPORTED) {
        const simjoin_status sq = check_matrix_args(ctx, Q, m, d);
        if (sq == SIMJOIN_ERR_ARG || st == SIMJOIN_OK) st = sq;
    }
    if (st != SIMJOIN_OK) return st;
    if (n + ctx->ioff >= SIMJOIN_MAX_ROWS || m + ctx->joff >= SIMJOIN_MAX_ROWS) return SIMJOIN_ERR_ARG;
    return SIMJOIN_OK;
}

bool encode_rows_map(const simjoin_ctx *ctx, CUtensorMap *map, const void *X, int64_t rows, int32_t d, int box_rows) {
    const size_t es = elem_size(ctx->dtype);
    const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)d * es};
    const cuuint32_t box[2] = {(cuuint32_t)(CHUNK_BYTES / es), (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapDataType dt = ctx->dtype == SIMJOIN_I8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    const CUresult r = ctx->encode(map, dt, 2, const_cast<void *>(X), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

template <bool kInt8>
cudaError_t launch_norms(const simjoin_ctx *ctx, const void *X, int64_t rows, int32_t d, int sqrt_out, void *norms,
                         void *minmax, unsigned int *all_max = nullptr) {
    using T = typename NormAcc<kInt8>::type;
    if (rows == 0) return cudaSuccess;
    const int g = (int)((size_t)d * elem_size(ctx->dtype) / 16);
    const unsigned blocks = (unsigned)((rows + NORM_TILE_ROWS - 1) / NORM_TILE_ROWS);
    row_norms_kernel<kInt8><<<blocks, NORM_THREADS, 0, ctx->stream>>>(reinterpret_cast<const uint4 *>(X), rows, g, sqrt_out,
                                                                     reinterpret_cast<T *>(norms), reinterpret_cast<T *>(minmax), all_max);
    return cudaGetLastError();
}

template <int DT, int KIND, bool ALT, int KC, bool GROUPED>
cudaError_t launch_join_kc(simjoin_ctx *ctx, const CUtensorMap &mp, const CUtensorMap &mq, const JoinParams &jp, int grid,
                           size_t smem) {
    auto kern = join_kernel<DT, KIND, ALT, KC, GROUPED>;
    if (!ctx->attr_set[DT][KIND][ALT ? 1 : 0][KC][GROUPED ? 1 : 0]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin);
        if (e != cudaSuccess) return e;
        ctx->attr_set[DT][KIND][ALT ? 1 : 0][KC][GROUPED ? 1 : 0] = true;
    }
    kern<<<grid, NUM_THREADS, smem, ctx->stream>>>(mp, mq, jp);
    return cudaGetLastError();
}

// Picks the instantiation with compile-time chunk count when the run-time parameters match it.
template <int DT, int KIND, bool ALT = false, bool GROUPED = false>
cudaError_t launch_join(simjoin_ctx *ctx, const CUtensorMap &mp, const CUtensorMap &mq, const JoinParams &jp, int grid,
                        size_t smem) {
    const bool fast = jp.stationary && jp.epi_release && jp.last_ksteps == 4;
    if (fast && jp.kc == 1 && jp.nstages == fast_nstages(1, p_bufs(GROUPED, 1)))
        return launch_join_kc<DT, KIND, ALT, 1, GROUPED>(ctx, mp, mq, jp, grid, smem);
    if (fast && jp.kc == 2 && jp.nstages == fast_nstages(2, p_bufs(GROUPED, 2)))
        return launch_join_kc<DT, KIND, ALT, 2, GROUPED>(ctx, mp, mq, jp, grid, smem);
    return launch_join_kc<DT, KIND, ALT, 0, GROUPED>(ctx, mp, mq, jp, grid, smem);
}

// The 16-epilogue-warp instantiations (dense outputs): bf16 kinds, rows of one or two whole chunks, brute-force schedule.
template <int DT, int KIND, bool ALT, int KC>
cudaError_t launch_join_dense_kc(simjoin_ctx *ctx, const CUtensorMap &mp, const CUtensorMap &mq, const JoinParams &jp, int grid, size_t smem) {
    constexpr int EW = 2 * NUM_EPI_WARPS;
    auto kern = join_kernel<DT, KIND, ALT, KC, false, GEO_STD, EW>;
    if (!ctx->attr_set_dense[KIND][ALT ? 1 : 0][KC]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin);
        if (e != cudaSuccess) return e;
        ctx->attr_set_dense[KIND][ALT ? 1 : 0][KC] = true;
    }
    kern<<<grid, num_threads(EW), smem, ctx->stream>>>(mp, mq, jp);
    return cudaGetLastError();
}
// Is there a dense instantiation for this geometry?
bool dense_available(bool i8, const JoinParams &jp) {
    const bool fast = jp.stationary && jp.epi_release && jp.last_ksteps == 4;
    return !i8 && fast && (jp.kc == 1 || jp.kc == 2) && jp.nstages == fast_nstages(jp.kc, p_bufs(false, jp.kc));
}
template <int KIND, bool ALT>
cudaError_t launch_join_dense(simjoin_ctx *ctx, const CUtensorMap &mp, const CUtensorMap &mq, const JoinParams &jp, int grid, size_t smem) {
    return jp.kc == 1 ? launch_join_dense_kc<DT_BF16, KIND, ALT, 1>(ctx, mp, mq, jp, grid, smem)
                      : launch_join_dense_kc<DT_BF16, KIND, ALT, 2>(ctx, mp, mq, jp, grid, smem);
}

// Chunks per row from which the join takes the long-row geometry.  Measured on B200 (n = m = 131 072, sustained,
// fraction of nominal): 384-byte rows 0.70 resident-P vs 0.61 long; 512-byte rows 0.56 vs 0.64; longer rows cannot
// keep P resident at all.
constexpr int LONG_MIN_KC = 4;
// The long-row geometry (256 x 256 tiles, nothing resident, one accumulator buffer): general join kinds only.
template <int DT, int KIND, bool ALT, bool GROUPED = false>
cudaError_t launch_join_long(simjoin_ctx *ctx, const CUtensorMap &mp, const CUtensorMap &mq, const JoinParams &jp, int grid,
                             size_t smem) {
    auto kern = join_kernel<DT, KIND, ALT, 0, GROUPED, GEO_LONG>;
    if (!ctx->attr_set_long[DT][KIND][ALT ? 1 : 0][GROUPED ? 1 : 0]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin);
        if (e != cudaSuccess) return e;
        ctx->attr_set_long[DT][KIND][ALT ? 1 : 0][GROUPED ? 1 : 0] = true;
    }
    kern<<<grid, NUM_THREADS, smem, ctx->stream>>>(mp, mq, jp);
    return cudaGetLastError();
}

// The wide-Q geometry of the store kind (one resident block of at most 128 rows against 256 streamed rows per tile).
cudaError_t launch_store_wideq(simjoin_ctx *ctx, const CUtensorMap &mp, const CUtensorMap &mq, const JoinParams &jp, int grid,
                               size_t smem) {
    auto kern = join_kernel<DT_BF16, KIND_STORE, false, 0, false, GEO_WIDEQ>;
    if (!ctx->attr_set_wideq) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin);
        if (e != cudaSuccess) return e;
        ctx->attr_set_wideq = true;
    }
    kern<<<grid, NUM_THREADS, smem, ctx->stream>>>(mp, mq, jp);
    return cudaGetLastError();
}

// Q tiles per panel.  A Q of up to 64 MiB is swept whole (it mostly stays in L2 and measured faster
// that way); a larger one is cut into panels of about 32 MiB that stay resident in L2 while every P
// block sweeps them (measured on a 128 MiB Q: 10.5 GB -> 0.74 GB of DRAM reads per launch).  Panels are
// balanced so that the last one is not a sliver.
int q_panel_tiles(int QT, int row_bytes, int tile_rows = TILE_N) {
    const long long tile_bytes = (long long)tile_rows * row_bytes;
    if ((long long)QT * tile_bytes <= (64LL << 20)) return QT;
    long long cap = (32LL << 20) / tile_bytes;
    if (cap < 8) cap = 8;
    const long long panels = (QT + cap - 1) / cap;
    return (int)((QT + panels - 1) / panels);
}

int clamp_to_i32(double v) {
    if (v >= 2147483647.0) return 2147483647;
    if (v <= -2147483648.0) return (-2147483647 - 1);
    return (int)v;
}

// Tile geometry of a join over rows of `row_bytes` bytes: chunks per tile, resident-P mode, ring depth,
// dynamic shared memory.  False when the ring would be too shallow.
bool tile_geometry(const simjoin_ctx *ctx, int64_t n, int64_t m, int row_bytes, size_t es, JoinParams &jp, size_t &smem,
                   bool grouped = false) {
    std::memset(&jp, 0, sizeof jp);
    jp.n = n;
    jp.m = m;
    jp.kc = (row_bytes + CHUNK_BYTES - 1) / CHUNK_BYTES;
    const int last_bytes = row_bytes - (jp.kc - 1) * CHUNK_BYTES;
    jp.last_ksteps = (last_bytes + 31) / 32;
    jp.elems_per_chunk = (int)(CHUNK_BYTES / es);
    jp.stationary = jp.kc <= MAX_STATIONARY_CHUNKS ? 1 : 0;
    const int p_bytes = jp.stationary ? p_bufs(grouped, jp.kc) * jp.kc * A_CHUNK_BYTES : 0;
    const int stage_bytes = B_CHUNK_BYTES + (jp.stationary ? 0 : A_CHUNK_BYTES);
    int nstages = (ctx->max_smem_optin - 1024 - CTRL_BYTES - STAGING_BYTES - p_bytes) / stage_bytes;
    if (nstages > MAX_STAGES) nstages = MAX_STAGES;
    if (nstages < 2) return false;
    jp.nstages = nstages;
    jp.epi_release = (jp.stationary && nstages >= 2 * jp.kc) ? 1 : 0;
    smem = 1024 + (size_t)p_bytes + (size_t)nstages * stage_bytes + STAGING_BYTES + CTRL_BYTES;
    return true;
}

// Thresholds in the precision each path decides in.
void set_thresholds(JoinParams &jp, bool i8, simjoin_kind kind, double threshold, int32_t d = 0) {
    jp.thr_d = threshold;
    if (i8) {
        if (kind == SIMJOIN_IP) jp.thr_i = clamp_to_i32(std::ceil(threshold));
        else if (kind == SIMJOIN_COS) jp.thr_f = (float)threshold;      // fp32 filter; the exact test takes thr_d
        else {
            const double r2 = std::floor(threshold * threshold);
            jp.thr_i = r2 >= 1073741824.0 ? 1073741824 : (int)r2;   // 2^30 exceeds every int8 squared distance here
        }
    } else {
        jp.thr_f = kind == SIMJOIN_L2 ? (float)(threshold * threshold) : (float)threshold;
        // a cosine lies in [-1, 1]: thresholds beyond +-2 decide like +-2, and the products t |x| |y| stay finite
        // (t = -inf times the norm 0 of a zero vector would be NaN, and its pairs would be lost)
        if (kind == SIMJOIN_COS) jp.thr_f = fminf(fmaxf(jp.thr_f, -2.f), 2.f);
        // the inner-product and cosine tests read the sign of s - b: with t = -0 a score of either zero gives +0 and passes
        if (kind != SIMJOIN_L2 && jp.thr_f == 0.f) jp.thr_f = -0.0f;
        if (kind != SIMJOIN_L2 && d > 0) {
            // Rounding error of the fp32-accumulated inner product relative to |x| |y| (sum |x_k y_k| is at most that),
            // charged like the Euclidean form below: d / 2 roundings of 2^-24 for the tensor core, 8 ceil(g / 32) + 5
            // for the norms the cosine test multiplies with, 16 for the epilogue's own operations.  Where this exceeds
            // half the tolerance band 1e-2 |t| the join decides its candidates from the rows in fp64 (see run_device).
            const int g = d * 2 / 16;
            jp.sel_coef = (float)std::ldexp(8.0 * ((g + 31) / 32) + 5.0 + 0.5 * d + 16.0, -24);
        }
        if (kind == SIMJOIN_L2 && d > 0) {
            // Rounding error of the norm expansion |x|^2 + |y|^2 - 2<x,y> as the tile epilogue evaluates it, relative to
            // |x|^2 + |y|^2, counted in fp32 roundings of at most 2^-24 each: the pre-pass adds a row's squares in at
            // most 8 ceil(g / 32) + 5 steps (g = 16-byte words per row); the tensor core is charged two roundings of
            // 2^-23 per 16-coordinate step on sum |x_k y_k| <= (|x|^2 + |y|^2) / 2, twice over (2<x,y>) and doubled once
            // more for what is not known of its internal order: d / 2; the epilogue's own operations and the
            // filter's coefficients: 16.  Measured errors are about a tenth of this.
            const int g = d * 2 / 16;
            const double roundings = 8.0 * ((g + 31) / 32) + 5.0 + 0.5 * d + 16.0;
            const double eps = std::ldexp(roundings, -24);
            jp.sel_coef = (float)eps;
            jp.l2_xscale = (float)(1.0 - eps);
            jp.l2_ycoef = (float)(0.5 * (1.0 - eps));
            // the difference form's own error (about d 2^-24 relative) is far inside the 2^-10 added here
            jp.l2_thr_filter = std::nextafterf((float)(threshold * threshold * (1.0 + 1.0 / 1024.0)), INFINITY);
            // ... and the mirror image: a score above the bound built from these passes whatever its rounding error
            // (|x|^2 + |y|^2 - 2s, raised by the error bound, is below r^2 (1 - 2^-10)), so its rows are not read
            jp.l2_xscale_hi = (float)(1.0 + eps);
            jp.l2_ycoef_hi = (float)(0.5 * (1.0 + eps));
            jp.l2_thr_sure = std::nextafterf((float)(threshold * threshold * (1.0 - 1.0 / 1024.0)), -INFINITY);
        }
    }
}

// What the norm pre-pass stores per row.  0: |x|^2; 1: |x| in fp32 (cosine); 2: the same with +inf for a zero
// vector -- cosine with t > 0, where a zero vector passes nothing: the epilogue's products t |x| |y| are then +inf.
int norm_mode(bool /*i8*/, simjoin_kind kind, float thr_f) {
    if (kind != SIMJOIN_COS) return 0;
    return thr_f > 0.f ? 2 : 1;                   // decided on the fp32 threshold the epilogue uses
}

// The inner-product kernel of launch_embedded: 16 epilogue warps, KC chunks per row, LASTK K steps in the last one.
template <int KC, int LASTK>
cudaError_t launch_embedded_kc(simjoin_ctx *ctx, const CUtensorMap &mp, const CUtensorMap &mq, const JoinParams &jp, int grid, size_t smem) {
    constexpr int EW = 2 * NUM_EPI_WARPS;
    auto kern = join_kernel<DT_BF16, KIND_IP, true, KC, false, GEO_STD, EW, LASTK>;      // threshold 0: sign test
    if (!ctx->attr_set_embed[KC][LASTK]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin);
        if (e != cudaSuccess) return e;
        ctx->attr_set_embed[KC][LASTK] = true;
    }
    kern<<<grid, num_threads(EW), smem, ctx->stream>>>(mp, mq, jp);
    return cudaGetLastError();
}

// A dense bf16 join through the operand transforms of embed_rows_kernel: both point sets are copied with 8 coordinates
// appended (context-owned buffers), and the 16-epilogue-warp sign-test kernel runs on the copies: <x', y'> >= 0.  For the
// Euclidean kind this is the plain form (the small-radius form stays on the points themselves; the selection words
// decide).  The copies' rows are padded with zeros to whole 128-byte chunks, so the whole-chunk instantiations apply and
// every box row is an aligned line.  Returns ERR_UNSUPPORTED (nothing launched) when the transformed rows do not fit
// two chunks or the threshold is not finite.  `jp_l2`: the join's own parameters (norms already computed).
simjoin_status launch_embedded(simjoin_ctx *ctx, simjoin_kind kind, const void *P, int64_t n, const void *Q, int64_t m, int32_t d,
                               const JoinScratch &scr, const JoinParams &jp_l2, int grid) {
    if ((d + 8) * 2 > 2 * CHUNK_BYTES || !std::isfinite(jp_l2.thr_f)) return SIMJOIN_ERR_UNSUPPORTED;
    const int row_bytes = ((d + 8) * 2 + CHUNK_BYTES - 1) / CHUNK_BYTES * CHUNK_BYTES, de = row_bytes / 2;      // whole chunks
    JoinParams jp;
    size_t smem = 0;
    if (!tile_geometry(ctx, n, m, row_bytes, 2, jp, smem)) return SIMJOIN_ERR_UNSUPPORTED;
    if (!dense_available(false, jp)) return SIMJOIN_ERR_UNSUPPORTED;
    if (!grow(ctx->emb_p, (size_t)n * row_bytes) || !grow(ctx->emb_q, (size_t)m * row_bytes)) return SIMJOIN_ERR_CUDA;
    const int g = d * 2 / 16, gout = row_bytes / 16;
    const int mode = kind == SIMJOIN_L2 ? EMBED_L2 : (kind == SIMJOIN_IP ? EMBED_IP : EMBED_COS);
    embed_rows_kernel<<<(unsigned)(((long long)n * gout + 255) / 256), 256, 0, ctx->stream>>>(
        reinterpret_cast<const uint4 *>(P), reinterpret_cast<const float *>(scr.nx), n, g, gout, mode, 0, jp_l2.thr_f, reinterpret_cast<uint4 *>(ctx->emb_p.ptr));
    embed_rows_kernel<<<(unsigned)(((long long)m * gout + 255) / 256), 256, 0, ctx->stream>>>(
        reinterpret_cast<const uint4 *>(Q), reinterpret_cast<const float *>(scr.ny), m, g, gout, mode, 1, 0.f, reinterpret_cast<uint4 *>(ctx->emb_q.ptr));
    if (cudaGetLastError() != cudaSuccess) return SIMJOIN_ERR_CUDA;
    jp.PB = jp_l2.PB;
    jp.QT = jp_l2.QT;
    jp.qpanel = q_panel_tiles(jp.QT, row_bytes, TILE_N);
    jp.out = jp_l2.out;
    jp.capacity = jp_l2.capacity;
    jp.counter = jp_l2.counter;
    jp.status = jp_l2.status;
    jp.ioff = jp_l2.ioff;
    jp.joff = jp_l2.joff;
    jp.zero_next = jp_l2.zero_next;
    jp.host_result = jp_l2.host_result;
    jp.done_ticket = jp_l2.done_ticket;
    jp.sel_mode = jp_l2.sel_mode;               // runs only when the selection words call for the plain form
    jp.sel_words = jp_l2.sel_words;
    jp.sel_coef = jp_l2.sel_coef;
    jp.sel_r2 = jp_l2.sel_r2;
    jp.thr_f = -0.0f;                           // <x', y'> >= 0 (Euclidean: (r^2 - |x - y|^2) / 2): a score of either zero passes
    jp.thr_d = 0.0;
    CUtensorMap mapP, mapQ;
    if (!encode_rows_map(ctx, &mapP, ctx->emb_p.ptr, n, de, P_ROWS) || !encode_rows_map(ctx, &mapQ, ctx->emb_q.ptr, m, de, TILE_N))
        return SIMJOIN_ERR_CUDA;
    // 32-byte K steps that the d + 8 coordinates reach into the last chunk: the issuers stop there
    const int lastk = ((d + 8) * 2 - (jp.kc - 1) * CHUNK_BYTES + 31) / 32;
    cudaError_t e = cudaErrorInvalidValue;
#define SJ_EMBED(KC_, LK_) e = launch_embedded_kc<KC_, LK_>(ctx, mapP, mapQ, jp, grid, smem)
    if (jp.kc == 1) { if (lastk == 1) SJ_EMBED(1, 1); else if (lastk == 2) SJ_EMBED(1, 2); else if (lastk == 3) SJ_EMBED(1, 3); else SJ_EMBED(1, 4); }
    else { if (lastk == 1) SJ_EMBED(2, 1); else if (lastk == 2) SJ_EMBED(2, 2); else if (lastk == 3) SJ_EMBED(2, 3); else SJ_EMBED(2, 4); }
#undef SJ_EMBED
    return e == cudaSuccess ? SIMJOIN_OK : SIMJOIN_ERR_CUDA;
}

// One launch of the brute-force join kernel in the geometry the rows call for.
template <int DT, int KIND, bool ALT>
cudaError_t launch_geo(simjoin_ctx *ctx, bool longk, const CUtensorMap &mp, const CUtensorMap &mq, const JoinParams &jp, int grid,
                       size_t smem) {
    return longk ? launch_join_long<DT, KIND, ALT>(ctx, mp, mq, jp, grid, smem) : launch_join<DT, KIND, ALT>(ctx, mp, mq, jp, grid, smem);
}
// Both variants back to back: each reads the selection words and only the one they call for does the work.
template <int DT, int KIND>
cudaError_t launch_both(simjoin_ctx *ctx, bool longk, const CUtensorMap &mp, const CUtensorMap &mq, const JoinParams &jp, int grid,
                        size_t smem) {
    const cudaError_t e = launch_geo<DT, KIND, false>(ctx, longk, mp, mq, jp, grid, smem);
    return e != cudaSuccess ? e : launch_geo<DT, KIND, true>(ctx, longk, mp, mq, jp, grid, smem);
}

// Which variant of the join kernel runs is decided on the device from two words of the control block that a pre-pass
// fills: int8 -- max|P|, max|Q| (the 16-bit epilogue when every score provably fits); bf16 Euclidean -- the largest
// squared norms (candidates decided from the rows when r^2 is below what the norm expansion resolves).
void set_selection(JoinParams &jp, bool i8, simjoin_kind kind, unsigned long long *d_ctrl) {
    if (i8) {
        jp.sel_mode = SEL_I8_RANGE;
        jp.sel_words = reinterpret_cast<const unsigned int *>(d_ctrl + 2);
    } else if (kind == SIMJOIN_L2) {
        jp.sel_mode = SEL_L2_RADIUS;
        jp.sel_words = reinterpret_cast<const unsigned int *>(d_ctrl + 3);
        jp.sel_r2 = jp.thr_f;
    }
}

// bf16 inner-product and cosine joins whose threshold sits so close to zero that the tolerance band 1e-2 |t| is narrower
// than the fp32 accumulation error of the tile product decide their candidates from the rows in fp64.
// Cosine: relative to |x| |y| both sides of the comparison scale alike, so the host can tell -- returns true and lowers the
// tile test's threshold to the filter's.
bool cos_row_form(JoinParams &jp, bool i8, simjoin_kind kind) {
    if (i8 || kind != SIMJOIN_COS) return false;
    const bool rows = jp.sel_coef > IPCOS_BAND_SHARE * std::fabs(jp.thr_f);
    if (rows) {
        jp.thr_hi = std::nextafterf(jp.thr_f + IPCOS_FILTER_MARGIN * jp.sel_coef, INFINITY);
        jp.thr_f = std::nextafterf(jp.thr_f - IPCOS_FILTER_MARGIN * jp.sel_coef, -INFINITY);
        if (jp.thr_f == 0.f) jp.thr_f = -0.0f;
    }
    return rows;
}
// Inner product: it depends on the largest norms, which the norm pre-pass leaves in the control block: the device chooses
// between the two forms (both are launched).
void ip_form_selection(JoinParams &jp, bool i8, simjoin_kind kind, unsigned long long *d_ctrl) {
    if (i8 || kind != SIMJOIN_IP) return;
    jp.sel_mode = SEL_IP_SMALL;
    jp.sel_words = reinterpret_cast<const unsigned int *>(d_ctrl + 3);
    jp.sel_r2 = jp.thr_f;
}

cudaError_t launch_maxabs(const simjoin_ctx *ctx, const void *P, long long p16, const void *Q, long long q16, unsigned long long *d_ctrl) {
    maxabs_i8_kernel<<<ctx->num_sms * 8, 256, 0, ctx->stream>>>(reinterpret_cast<const uint4 *>(P), p16, reinterpret_cast<const uint4 *>(Q), q16,
                                                                 reinterpret_cast<unsigned int *>(d_ctrl + 2));
    return cudaGetLastError();
}

// The join on device buffers.  Arguments were validated by the caller.  `fixed`: working memory provided by the caller
// (the allocation-free entry point); otherwise the context's buffers are grown to fit.  No host round trip happens
// between the pre-passes and the join: one stream synchronisation at the end.
simjoin_status run_device(simjoin_ctx *ctx, const void *P, int64_t n, const void *Q, int64_t m, int32_t d,
                          simjoin_kind kind, double threshold, int32_t *out_pairs, uint64_t capacity, uint64_t *count,
                          const JoinScratch *fixed = nullptr) {
    *count = 0;
    ctx->have_timing = false;
    if (n == 0 || m == 0) return SIMJOIN_OK;
    const bool i8 = ctx->dtype == SIMJOIN_I8;
    const size_t es = elem_size(ctx->dtype);
    const int row_bytes = (int)(d * es);

    JoinParams jp;
    size_t smem = 0;
    if (!tile_geometry(ctx, n, m, row_bytes, es, jp, smem)) return SIMJOIN_ERR_UNSUPPORTED;
    // rows of 512 bytes and more take the long-row geometry
    const bool longk = jp.kc >= LONG_MIN_KC;
    const int tn = longk ? LONG_TN : TILE_N;
    if (longk) {
        jp.stationary = 0;
        jp.epi_release = 0;
        jp.nstages = LONG_STAGES;
        smem = 1024 + (size_t)LONG_STAGES * LONG_STAGE_BYTES + STAGING_BYTES + CTRL_BYTES;
        if (smem > (size_t)ctx->max_smem_optin) return SIMJOIN_ERR_UNSUPPORTED;
        // one P tile per CTA plus a Q panel must fit in L2 (126 MB) for the sweep schedule; beyond that, 2-D waves
        if ((long long)ctx->num_sms * P_ROWS * row_bytes > (48LL << 20) && ctx->num_sms >= 8) jp.wave_gq = 4;
    }
    // A context without history (no join yet) that is about to run a large bf16 join which has a dense layout first
    // counts the pairs of a sample -- the first P tile against one Q tile per SM, a few microseconds -- so that its
    // first join already runs in the layout its output density calls for (the count sets last_density).
    if (!fixed && !i8 && !longk && ctx->dense_mode == 2 && ctx->last_density < 0.0 && dense_available(i8, jp) &&
        2.0 * (double)n * (double)m * (double)d >= DENSITY_SAMPLE_MIN_OPS) {
        ctx->last_density = 0.0;                // the sample itself runs sparse
        uint64_t sampled = 0;
        const simjoin_status ss = run_device(ctx, P, std::min<int64_t>(n, P_ROWS), Q, std::min<int64_t>(m, (int64_t)ctx->num_sms * TILE_N), d, kind,
                                             threshold, nullptr, 0, &sampled);
        if (ss != SIMJOIN_OK && ss != SIMJOIN_ERR_CAPACITY) return ss;
        ctx->have_timing = false;
    }
    jp.PB = (int)((n + P_ROWS - 1) / P_ROWS);
    jp.QT = (int)((m + tn - 1) / tn);
    jp.qpanel = q_panel_tiles(jp.QT, row_bytes, tn);
    jp.out = reinterpret_cast<int2 *>(out_pairs);
    jp.capacity = capacity;
    jp.ioff = (int)ctx->ioff;
    jp.joff = (int)ctx->joff;

    set_thresholds(jp, i8, kind, threshold, d);
    jp.rows_p = P;
    jp.rows_q = Q;
    jp.row_bytes = row_bytes;

    // bf16 inner-product joins run the norm pre-pass for its maxima: they tell whether the threshold's tolerance band is
    // wider than the fp32 accumulation error (decided on the device, like the Euclidean form)
    const bool need_norms = kind != SIMJOIN_IP || !i8;
    // bf16 cosine with a threshold that close to zero: the tile test becomes a filter lowered by the error bound and every
    // candidate is decided from its rows in fp64 (relative to |x| |y| both sides of the comparison scale alike, so the
    // host can tell)
    const bool cos_rows = cos_row_form(jp, i8, kind);
    JoinScratch scr;
    if (fixed) {
        scr = *fixed;
    } else {
        // ny is read in 16-entry groups up to the end of the last Q tile: pad it to whole tiles
        if (need_norms && (!grow(ctx->nx, (size_t)n * 4) || !grow(ctx->ny, (size_t)jp.QT * tn * 4) || !grow(ctx->qstat, (size_t)jp.QT * 8)))
            return SIMJOIN_ERR_CUDA;
        scr = JoinScratch{ctx->nx.ptr, ctx->ny.ptr, ctx->qstat.ptr, ctx->d_ctrl, ctx->h_ctrl, true};
    }
    // The context owns two control blocks and alternates between them: the join kernel of one call zeroes the block of
    // the next, which then starts without a memset (one step less in the stream's dependent chain; it shows on small
    // joins).  A call that fails, or any other entry point that uses the control block, breaks the chain, and the next
    // call clears its block itself.
    bool need_clear = true;
    int cur = 0;
    if (!fixed) {
        if (ctx->ctrl_clean >= 0) {
            cur = ctx->ctrl_clean;
            need_clear = false;
        }
        scr.d_ctrl = ctx->d_ctrl + 8 * cur;
        jp.zero_next = ctx->d_ctrl + 8 * (cur ^ 1);
        ctx->ctrl_clean = -1;
    }
    jp.counter = scr.d_ctrl;
    jp.status = reinterpret_cast<unsigned int *>(scr.d_ctrl + 1);
    if (scr.h_ctrl_mapped) {
        jp.host_result = scr.h_ctrl;
        jp.done_ticket = reinterpret_cast<unsigned int *>(scr.d_ctrl + 4);
    }
    if (need_norms) {
        jp.nx = scr.nx;
        jp.ny = scr.ny;
        jp.qstat = scr.qstat;
    }
    // small int8 joins take the 32-bit epilogue unasked (see DEFAULT_SELECT_MIN_OPS)
    const bool select_i8 = i8 && 2.0 * (double)n * (double)m * (double)d >= ctx->select_min_ops;
    if (!i8 || select_i8) set_selection(jp, i8, kind, scr.d_ctrl);
    ip_form_selection(jp, i8, kind, scr.d_ctrl);

    CUtensorMap mapP, mapQ;
    if (!encode_rows_map(ctx, &mapP, P, n, d, P_ROWS) || !encode_rows_map(ctx, &mapQ, Q, m, d, tn))
        return SIMJOIN_ERR_CUDA;

    cudaStream_t s = ctx->stream;
    const bool timed = ctx->ev[0] != nullptr && ctx->kernel_timing;
    // the control block keeps the previous call's contents: counter, status and selection words start at zero
    if (need_clear && cudaMemsetAsync(scr.d_ctrl, 0, 64, s) != cudaSuccess) return SIMJOIN_ERR_CUDA;
    if (select_i8 && launch_maxabs(ctx, P, (long long)n * row_bytes / 16, Q, (long long)m * row_bytes / 16, scr.d_ctrl) != cudaSuccess)
        return SIMJOIN_ERR_CUDA;
    if (timed && need_norms) cudaEventRecord(ctx->ev[0], s);      // (every event is a step in the stream: none without a pre-pass)
    if (need_norms) {
        const int sq = norm_mode(i8, kind, i8 ? (float)threshold : jp.thr_f);
        unsigned int *nmax = (!i8 && kind != SIMJOIN_COS) ? reinterpret_cast<unsigned int *>(scr.d_ctrl + 3) : nullptr;
        cudaError_t e1, e2;
        if (i8) {
            e1 = launch_norms<true>(ctx, P, n, d, sq, scr.nx, nullptr);
            e2 = launch_norms<true>(ctx, Q, m, d, sq, scr.ny, scr.qstat);
        } else {
            e1 = launch_norms<false>(ctx, P, n, d, sq, scr.nx, nullptr, nmax);
            e2 = launch_norms<false>(ctx, Q, m, d, sq, scr.ny, scr.qstat, nmax ? nmax + 1 : nullptr);
        }
        if (e1 != cudaSuccess || e2 != cudaSuccess) return SIMJOIN_ERR_CUDA;
        // the padding of ny up to whole tiles is read (and masked) by the epilogue: keep it defined
        const size_t pad = (size_t)jp.QT * tn - (size_t)m;
        if (pad > 0 && cudaMemsetAsync(static_cast<char *>(scr.ny) + (size_t)m * 4, 0, pad * 4, s) != cudaSuccess) return SIMJOIN_ERR_CUDA;
    }
    if (timed) cudaEventRecord(ctx->ev[1], s);
    const int grid = ctx->num_sms;
    cudaError_t e = cudaErrorInvalidValue;
    const char *layout = "8 epilogue warps";
    if (i8 && !select_i8) {
        if (kind == SIMJOIN_IP) e = launch_geo<DT_I8, KIND_IP, false>(ctx, longk, mapP, mapQ, jp, grid, smem);
        else if (kind == SIMJOIN_L2) e = launch_geo<DT_I8, KIND_L2, false>(ctx, longk, mapP, mapQ, jp, grid, smem);
        else e = launch_geo<DT_I8, KIND_COS, false>(ctx, longk, mapP, mapQ, jp, grid, smem);
    } else if (i8 && kind == SIMJOIN_IP) e = launch_both<DT_I8, KIND_IP>(ctx, longk, mapP, mapQ, jp, grid, smem);
    else if (i8 && kind == SIMJOIN_L2) e = launch_both<DT_I8, KIND_L2>(ctx, longk, mapP, mapQ, jp, grid, smem);
    else if (i8 && kind == SIMJOIN_COS) e = launch_both<DT_I8, KIND_COS>(ctx, longk, mapP, mapQ, jp, grid, smem);
    else if (cos_rows) e = launch_geo<DT_BF16, KIND_COS, true>(ctx, longk, mapP, mapQ, jp, grid, smem);
    else if (!i8 && dense_available(i8, jp) && !longk &&
             (ctx->dense_mode == 1 || (ctx->dense_mode == 2 && ctx->last_density >= DENSE_MIN_PAIRS_PER_BLOCK))) {
        // The last join on this context was dense: the 16-epilogue-warp instantiation of the same kind -- or, where the
        // transformed rows still fit two chunks, the sign test on transformed operands (Section 4's ip-distance
        // embeddings: embed_rows_kernel).  Euclidean joins: that is the plain form; the small-radius form stays on
        // the points themselves, and whichever the selection words call for does the work.
        const bool embed = !fixed && (ctx->dense_mode == 1 || ctx->last_density >= EMBED_MIN_PAIRS_PER_BLOCK);
        const simjoin_status es2 = embed ? launch_embedded(ctx, kind, P, n, Q, m, d, scr, jp, grid) : SIMJOIN_ERR_UNSUPPORTED;
        if (es2 == SIMJOIN_ERR_CUDA) return SIMJOIN_ERR_CUDA;
        layout = es2 == SIMJOIN_OK ? "16 epilogue warps on transformed operands" : "16 epilogue warps";
        e = cudaSuccess;
        if (kind == SIMJOIN_IP) {
            if (es2 != SIMJOIN_OK) e = launch_join_dense<KIND_IP, false>(ctx, mapP, mapQ, jp, grid, smem);
            // (the row-deciding form of the inner-product join has one layout: 8 epilogue warps)
            if (e == cudaSuccess) e = launch_geo<DT_BF16, KIND_IP, true>(ctx, false, mapP, mapQ, jp, grid, smem);
        }
        else if (kind == SIMJOIN_COS) { if (es2 != SIMJOIN_OK) e = launch_join_dense<KIND_COS, false>(ctx, mapP, mapQ, jp, grid, smem); }
        else {
            if (es2 != SIMJOIN_OK) e = launch_join_dense<KIND_L2, false>(ctx, mapP, mapQ, jp, grid, smem);
            if (e == cudaSuccess) e = launch_join_dense<KIND_L2, true>(ctx, mapP, mapQ, jp, grid, smem);
        }
    }
    else if (!i8 && kind == SIMJOIN_IP) e = launch_both<DT_BF16, KIND_IP>(ctx, longk, mapP, mapQ, jp, grid, smem);
    else if (!i8 && kind == SIMJOIN_COS) e = launch_geo<DT_BF16, KIND_COS, false>(ctx, longk, mapP, mapQ, jp, grid, smem);
    else if (!i8 && kind == SIMJOIN_L2) e = launch_both<DT_BF16, KIND_L2>(ctx, longk, mapP, mapQ, jp, grid, smem);
    if (e != cudaSuccess) return SIMJOIN_ERR_CUDA;
    if (timed) cudaEventRecord(ctx->ev[2], s);
    if (!scr.h_ctrl_mapped && cudaMemcpyAsync(scr.h_ctrl, scr.d_ctrl, 16, cudaMemcpyDeviceToHost, s) != cudaSuccess) return SIMJOIN_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) {
        cudaGetLastError();
        return SIMJOIN_ERR_CUDA;
    }
    const unsigned int kstatus = (unsigned int)(scr.h_ctrl[1] & 0xffffffffu);
    if (kstatus != 0) return SIMJOIN_ERR_TIMEOUT;
    if (!fixed) ctx->ctrl_clean = cur ^ 1;        // the kernel has zeroed the other block
    *count = scr.h_ctrl[0];
    if (debug_log())
        std::fprintf(stderr, "[simjoin] run dtype=%s kind=%d n=%lld m=%lld d=%d t=%g: %d chunk(s) per row, %s geometry, %d ring stages, %s, "
                             "%s, pairs=%llu capacity=%llu\n",
                     i8 ? "i8" : "bf16", (int)kind, (long long)n, (long long)m, (int)d, threshold, jp.kc,
                     longk ? (jp.wave_gq ? "long-row (2-D waves)" : "long-row") : (jp.stationary ? "resident-P" : "streamed"), jp.nstages, layout,
                     cos_rows ? "candidates decided from the rows (threshold near zero)"
                     : jp.sel_mode == SEL_NONE ? "one variant"
                     : jp.sel_mode == SEL_I8_RANGE ? "epilogue width chosen on the device"
                     : jp.sel_mode == SEL_IP_SMALL ? "plain or row-deciding form chosen on the device"
                                                   : "Euclidean form chosen on the device",
                     (unsigned long long)*count, (unsigned long long)capacity);
    ctx->last_density = (double)*count / ((double)((n + 31) / 32) * (double)((m + 127) / 128));
    float a = 0.f, b = 0.f;
    if (timed && (!need_norms || cudaEventElapsedTime(&a, ctx->ev[0], ctx->ev[1]) == cudaSuccess) &&
        cudaEventElapsedTime(&b, ctx->ev[1], ctx->ev[2]) == cudaSuccess) {
        ctx->prepass_ms = need_norms ? a : 0.f;
        ctx->join_ms = b;
        ctx->have_timing = true;
    }
    return *count > capacity ? SIMJOIN_ERR_CAPACITY : SIMJOIN_OK;
}

// Hash keys of the hyperplane family for all rows of X: the tile kernel with the hyperplane matrix as the resident
// operand, the points as the streamed one and the sign-collecting epilogue; writes the key records.
template <int DT>
simjoin_status hyperplane_keys(simjoin_ctx *ctx, const void *planes, int plane_rows, const void *X, int64_t rows, int32_t d,
                               void *rec, int rec_words) {
    const size_t es = elem_size(ctx->dtype);
    JoinParams jp;
    size_t smem = 0;
    if (!tile_geometry(ctx, plane_rows, rows, (int)(d * es), es, jp, smem)) return SIMJOIN_ERR_UNSUPPORTED;
    jp.PB = (plane_rows + P_ROWS - 1) / P_ROWS;
    jp.QT = (int)((rows + TILE_N - 1) / TILE_N);
    jp.qpanel = jp.QT;                 // the points are read once per 256 hyperplanes: one long sweep per CTA
    jp.counter = ctx->d_ctrl;
    jp.status = reinterpret_cast<unsigned int *>(ctx->d_ctrl + 1);
    jp.key_out = reinterpret_cast<uint32_t *>(rec);
    jp.key_ld = (long long)rec_words * 4;
    CUtensorMap mapA, mapX;
    if (!encode_rows_map(ctx, &mapA, planes, plane_rows, d, P_ROWS) || !encode_rows_map(ctx, &mapX, X, rows, d, TILE_N)) return SIMJOIN_ERR_CUDA;
    auto kern = join_kernel<DT, KIND_SIGN, false, 0, false, GEO_STD>;
    if (!ctx->attr_set_sign[DT]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin) != cudaSuccess) return SIMJOIN_ERR_CUDA;
        ctx->attr_set_sign[DT] = true;
    }
    kern<<<ctx->num_sms, NUM_THREADS, smem, ctx->stream>>>(mapA, mapX, jp);
    return cudaGetLastError() == cudaSuccess ? SIMJOIN_OK : SIMJOIN_ERR_CUDA;
}

// One bucketed join launch: instantiation by element type, kind, variant and geometry.
cudaError_t launch_bucketed(simjoin_ctx *ctx, bool i8, simjoin_kind kind, bool longk, const CUtensorMap &mp,
                            const CUtensorMap &mq, const JoinParams &jp, size_t smem, bool cos_rows) {
    const int grid = ctx->num_sms;
#define SJ_BUCKETED(DT, KIND, ALT)                                                          \
    (longk ? launch_join_long<DT, KIND, ALT, true>(ctx, mp, mq, jp, grid, smem) \
           : launch_join<DT, KIND, ALT, true>(ctx, mp, mq, jp, grid, smem))
    // where the device selects the variant (int8; bf16 Euclidean and inner product) both are launched and one returns at
    // once; the row-deciding form of the bf16 cosine join is the host's choice (cos_rows)
#define SJ_BUCKETED_BOTH(DT, KIND)                                   \
    {                                                                \
        const cudaError_t e = SJ_BUCKETED(DT, KIND, false);          \
        return e != cudaSuccess ? e : SJ_BUCKETED(DT, KIND, true);   \
    }
    if (i8 && kind == SIMJOIN_IP) SJ_BUCKETED_BOTH(DT_I8, KIND_IP)
    if (i8 && kind == SIMJOIN_L2) SJ_BUCKETED_BOTH(DT_I8, KIND_L2)
    if (i8 && kind == SIMJOIN_COS) SJ_BUCKETED_BOTH(DT_I8, KIND_COS)
    if (!i8 && kind == SIMJOIN_IP) SJ_BUCKETED_BOTH(DT_BF16, KIND_IP)
    if (!i8 && kind == SIMJOIN_COS) return cos_rows ? SJ_BUCKETED(DT_BF16, KIND_COS, true) : SJ_BUCKETED(DT_BF16, KIND_COS, false);
    if (!i8 && kind == SIMJOIN_L2) SJ_BUCKETED_BOTH(DT_BF16, KIND_L2)
#undef SJ_BUCKETED_BOTH
#undef SJ_BUCKETED
    return cudaErrorInvalidValue;
}

simjoin_status lsh_device(simjoin_ctx *ctx, const void *P, int64_t n, const void *Q, int64_t m, int32_t d, simjoin_kind kind,
                          double threshold, simjoin_lsh_family family, int32_t L, int32_t L_low, int32_t k, uint64_t seed,
                          int32_t *out_pairs, uint64_t capacity, uint64_t *count) {
    *count = 0;
    ctx->have_timing = false;
    if (n == 0 || m == 0) return SIMJOIN_OK;
    const bool i8 = ctx->dtype == SIMJOIN_I8;
    const size_t es = elem_size(ctx->dtype);
    const int row_bytes = (int)(d * es);
    const bool need_norms = kind != SIMJOIN_IP || !i8;       // (bf16 inner product: for the maxima, as in run_device)

    JoinParams jp;
    size_t smem = 0;
    if (!tile_geometry(ctx, n, m, row_bytes, es, jp, smem, true)) return SIMJOIN_ERR_UNSUPPORTED;
    // rows of 512 bytes and more: the long-row geometry inside the buckets too
    const bool longk = jp.kc >= LONG_MIN_KC;
    if (longk) {
        jp.stationary = 0;
        jp.epi_release = 0;
        jp.nstages = LONG_STAGES;
        smem = 1024 + (size_t)LONG_STAGES * LONG_STAGE_BYTES + STAGING_BYTES + CTRL_BYTES;
        if (smem > (size_t)ctx->max_smem_optin) return SIMJOIN_ERR_UNSUPPORTED;
    }
    const int nb_max = 1 << k;
    const size_t max_units = (size_t)((n + P_ROWS - 1) / P_ROWS) + (size_t)nb_max;
    // misc: hist_p | hist_q | cursor_p | cursor_q (nb words each) | nunits (padded to 16 B) | units
    const size_t off_coords = ((size_t)4 * nb_max * 4 + 16 + 15) & ~(size_t)15;       // sampled coordinates: reps x k ints
    const size_t off_units = (off_coords + (size_t)LSH_MAX_REPS * LSH_MAX_BITS * 4 + 15) & ~(size_t)15;
    const int reps = L + L_low;
    const int rec_words = (reps + 7) / 8, stride = rec_words * 8;   // key record of a row: 16-bit keys, padded to 16 bytes
    const size_t rec_bytes = (size_t)rec_words * 16;
    if (!grow(ctx->lsh_keys_p, n * rec_bytes) || !grow(ctx->lsh_keys_q, m * rec_bytes) ||
        !grow(ctx->lsh_perm_p, (size_t)n * 4) || !grow(ctx->lsh_perm_q, (size_t)m * 4) ||
        !grow(ctx->lsh_sorted_p, (size_t)n * row_bytes) || !grow(ctx->lsh_sorted_q, (size_t)m * row_bytes) ||
        !grow(ctx->lsh_misc, off_units + max_units * 16))
        return SIMJOIN_ERR_CUDA;
    // row terms of the regrouped rows (norm kinds); a bucket's last tile may read up to a tile past the end of ny
    const size_t ny_entries = (size_t)m + LONG_TN + 8;
    if (need_norms && (!grow(ctx->nx, (size_t)n * 4) || !grow(ctx->ny, ny_entries * 4) ||
                       !grow(ctx->qstat, (size_t)((m + NORM_TILE_ROWS - 1) / NORM_TILE_ROWS) * 8)))
        return SIMJOIN_ERR_CUDA;
    unsigned int *hist_p = reinterpret_cast<unsigned int *>(ctx->lsh_misc.ptr);
    unsigned int *hist_q = hist_p + nb_max, *cursor_p = hist_q + nb_max, *cursor_q = cursor_p + nb_max, *nunits = cursor_q + nb_max;
    int4 *units = reinterpret_cast<int4 *>(reinterpret_cast<unsigned char *>(ctx->lsh_misc.ptr) + off_units);
    int *coords = reinterpret_cast<int *>(reinterpret_cast<unsigned char *>(ctx->lsh_misc.ptr) + off_coords);
    uint16_t *keys_p = reinterpret_cast<uint16_t *>(ctx->lsh_keys_p.ptr), *keys_q = reinterpret_cast<uint16_t *>(ctx->lsh_keys_q.ptr);
    int *perm_p = reinterpret_cast<int *>(ctx->lsh_perm_p.ptr), *perm_q = reinterpret_cast<int *>(ctx->lsh_perm_q.ptr);

    jp.out = reinterpret_cast<int2 *>(out_pairs);
    jp.capacity = capacity;
    jp.counter = ctx->d_ctrl;
    jp.status = reinterpret_cast<unsigned int *>(ctx->d_ctrl + 1);
    jp.ioff = (int)ctx->ioff;
    jp.joff = (int)ctx->joff;
    set_thresholds(jp, i8, kind, threshold, d);
    set_selection(jp, i8, kind, ctx->d_ctrl);
    const bool cos_rows = cos_row_form(jp, i8, kind);
    ip_form_selection(jp, i8, kind, ctx->d_ctrl);
    jp.rows_p = ctx->lsh_sorted_p.ptr;      // the regrouped rows, addressed by regrouped position
    jp.rows_q = ctx->lsh_sorted_q.ptr;
    jp.row_bytes = row_bytes;
    if (need_norms) {
        jp.nx = ctx->nx.ptr;
        jp.ny = ctx->ny.ptr;
        jp.qstat = ctx->qstat.ptr;
    }
    jp.units = units;
    jp.nunits = nunits;
    jp.perm_p = perm_p;
    jp.perm_q = perm_q;
    jp.rec_p = reinterpret_cast<const uint4 *>(ctx->lsh_keys_p.ptr);      // in the rows' original order
    jp.rec_q = reinterpret_cast<const uint4 *>(ctx->lsh_keys_q.ptr);
    jp.rec_words = rec_words;

    CUtensorMap mapP, mapQ;
    if (!encode_rows_map(ctx, &mapP, ctx->lsh_sorted_p.ptr, n, d, P_ROWS) ||
        !encode_rows_map(ctx, &mapQ, ctx->lsh_sorted_q.ptr, m, d, longk ? LONG_TN : TILE_N))
        return SIMJOIN_ERR_CUDA;

    cudaStream_t s = ctx->stream;
    ctx->ctrl_clean = -1;                         // this call uses the first control block and leaves it dirty
    if (cudaMemsetAsync(ctx->d_ctrl, 0, 64, s) != cudaSuccess) return SIMJOIN_ERR_CUDA;
    // the variant (16-bit epilogue for int8, row-decided candidates for small bf16 radii) is selected on the device, as in
    // the brute-force join; the norm kinds' pre-pass runs once per repetition on the regrouped rows and folds the same
    // maxima into the selection words every time
    if (i8 && launch_maxabs(ctx, P, (long long)n * d / 16, Q, (long long)m * d / 16, ctx->d_ctrl) != cudaSuccess) return SIMJOIN_ERR_CUDA;
    if (need_norms && cudaMemsetAsync(static_cast<char *>(ctx->ny.ptr) + (size_t)m * 4, 0, (ny_entries - (size_t)m) * 4, s) != cudaSuccess)
        return SIMJOIN_ERR_CUDA;

    cudaEventRecord(ctx->ev[0], s);
    if (family == SIMJOIN_LSH_HYPERPLANES) {
        // all projections of all points at once: (points) x (16 rows per repetition, padded to whole key words)
        const int plane_rows = stride * 16;
        if (!grow(ctx->lsh_planes, (size_t)plane_rows * row_bytes)) return SIMJOIN_ERR_CUDA;
        const unsigned pblocks = (unsigned)(((long long)plane_rows * d + 255) / 256);
        simjoin_status hs;
        if (i8) {
            lsh_hyperplanes_kernel<<<pblocks, 256, 0, s>>>(seed, L, L_low, k, d, stride, reinterpret_cast<int8_t *>(ctx->lsh_planes.ptr));
            hs = hyperplane_keys<DT_I8>(ctx, ctx->lsh_planes.ptr, plane_rows, P, n, d, keys_p, rec_words);
            if (hs == SIMJOIN_OK) hs = hyperplane_keys<DT_I8>(ctx, ctx->lsh_planes.ptr, plane_rows, Q, m, d, keys_q, rec_words);
        } else {
            lsh_hyperplanes_kernel<<<pblocks, 256, 0, s>>>(seed, L, L_low, k, d, stride, reinterpret_cast<uint16_t *>(ctx->lsh_planes.ptr));
            hs = hyperplane_keys<DT_BF16>(ctx, ctx->lsh_planes.ptr, plane_rows, P, n, d, keys_p, rec_words);
            if (hs == SIMJOIN_OK) hs = hyperplane_keys<DT_BF16>(ctx, ctx->lsh_planes.ptr, plane_rows, Q, m, d, keys_q, rec_words);
        }
        if (hs != SIMJOIN_OK) return hs;
    } else {
        const unsigned bn = (unsigned)((n + LSH_KEYS_STAGED_ROWS - 1) / LSH_KEYS_STAGED_ROWS), bm = (unsigned)((m + LSH_KEYS_STAGED_ROWS - 1) / LSH_KEYS_STAGED_ROWS);
        const size_t sm = (size_t)LSH_KEYS_STAGED_ROWS * (row_bytes / 4 + 1) * 4;
        const bool staged = row_bytes <= LSH_KEYS_STAGED_MAX_D;
        lsh_coordinates_kernel<<<1, 64, 0, s>>>(seed, L + L_low, k, d, family == SIMJOIN_LSH_BITS ? 1 : 0, coords);
        if (i8) {
            const int8_t *p8 = reinterpret_cast<const int8_t *>(P), *q8 = reinterpret_cast<const int8_t *>(Q);
            if (staged) {
                lsh_keys_staged_kernel<<<bn, 256, sm, s>>>(p8, n, d, L, L_low, k, coords, keys_p, stride);
                lsh_keys_staged_kernel<<<bm, 256, sm, s>>>(q8, m, d, L, L_low, k, coords, keys_q, stride);
            } else {
                lsh_keys_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(p8, n, d, L, L_low, k, coords, keys_p, stride);
                lsh_keys_kernel<<<(unsigned)((m + 255) / 256), 256, 0, s>>>(q8, m, d, L, L_low, k, coords, keys_q, stride);
            }
        } else {
            const int16_t *p16 = reinterpret_cast<const int16_t *>(P), *q16 = reinterpret_cast<const int16_t *>(Q);
            if (staged) {
                lsh_keys_staged_kernel<<<bn, 256, sm, s>>>(p16, n, d, L, L_low, k, coords, keys_p, stride);
                lsh_keys_staged_kernel<<<bm, 256, sm, s>>>(q16, m, d, L, L_low, k, coords, keys_q, stride);
            } else {
                lsh_keys_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(p16, n, d, L, L_low, k, coords, keys_p, stride);
                lsh_keys_kernel<<<(unsigned)((m + 255) / 256), 256, 0, s>>>(q16, m, d, L, L_low, k, coords, keys_q, stride);
            }
        }
    }
    if (cudaGetLastError() != cudaSuccess) return SIMJOIN_ERR_CUDA;
    cudaEventRecord(ctx->ev[1], s);
    const int g = row_bytes / 16;
    const unsigned hist_blocks = (unsigned)ctx->num_sms * 4;
    const int rows_per_block = LSH_SORT_THREADS * LSH_SORT_ITEMS;
    for (int l = 0; l < reps; ++l) {
        const uint16_t *kp = keys_p + l, *kq = keys_q + l;          // column l of the key records
        const int nb = l < L ? nb_max : nb_max / 2;          // buckets of this repetition
        if (cudaMemsetAsync(hist_p, 0, (size_t)2 * nb_max * 4, s) != cudaSuccess) return SIMJOIN_ERR_CUDA;
        lsh_hist_kernel<<<hist_blocks, LSH_SORT_THREADS, 0, s>>>(kp, stride, n, nb, hist_p);
        lsh_hist_kernel<<<hist_blocks, LSH_SORT_THREADS, 0, s>>>(kq, stride, m, nb, hist_q);
        lsh_offsets_units_kernel<<<1, 1024, 0, s>>>(hist_p, hist_q, nb, cursor_p, cursor_q, units, nunits, P_ROWS);
        lsh_scatter_kernel<<<(unsigned)((n + rows_per_block - 1) / rows_per_block), LSH_SORT_THREADS, 0, s>>>(kp, stride, n, nb,
                                                                                                              cursor_p, perm_p);
        lsh_scatter_kernel<<<(unsigned)((m + rows_per_block - 1) / rows_per_block), LSH_SORT_THREADS, 0, s>>>(kq, stride, m, nb,
                                                                                                              cursor_q, perm_q);
        lsh_gather_rows_kernel<<<(unsigned)(((long long)n * g + 255) / 256), 256, 0, s>>>(
            reinterpret_cast<const uint4 *>(P), perm_p, n, g, reinterpret_cast<uint4 *>(ctx->lsh_sorted_p.ptr));
        lsh_gather_rows_kernel<<<(unsigned)(((long long)m * g + 255) / 256), 256, 0, s>>>(
            reinterpret_cast<const uint4 *>(Q), perm_q, m, g, reinterpret_cast<uint4 *>(ctx->lsh_sorted_q.ptr));
        if (need_norms) {
            // row terms and per-256-row bounds of the regrouped rows
            const int sq = norm_mode(i8, kind, i8 ? (float)threshold : jp.thr_f);
            cudaError_t e1, e2;
            if (i8) {
                e1 = launch_norms<true>(ctx, ctx->lsh_sorted_p.ptr, n, d, sq, ctx->nx.ptr, nullptr);
                e2 = launch_norms<true>(ctx, ctx->lsh_sorted_q.ptr, m, d, sq, ctx->ny.ptr, ctx->qstat.ptr);
            } else {
                unsigned int *nmax = kind != SIMJOIN_COS ? reinterpret_cast<unsigned int *>(ctx->d_ctrl + 3) : nullptr;
                e1 = launch_norms<false>(ctx, ctx->lsh_sorted_p.ptr, n, d, sq, ctx->nx.ptr, nullptr, nmax);
                e2 = launch_norms<false>(ctx, ctx->lsh_sorted_q.ptr, m, d, sq, ctx->ny.ptr, ctx->qstat.ptr, nmax ? nmax + 1 : nullptr);
            }
            if (e1 != cudaSuccess || e2 != cudaSuccess) return SIMJOIN_ERR_CUDA;
        }
        if (cudaGetLastError() != cudaSuccess) return SIMJOIN_ERR_CUDA;
        jp.rep = l;
        if (launch_bucketed(ctx, i8, kind, longk, mapP, mapQ, jp, smem, cos_rows) != cudaSuccess) return SIMJOIN_ERR_CUDA;
    }
    cudaEventRecord(ctx->ev[2], s);
    if (cudaMemcpyAsync(ctx->h_ctrl, ctx->d_ctrl, 16, cudaMemcpyDeviceToHost, s) != cudaSuccess) return SIMJOIN_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) {
        cudaGetLastError();
        return SIMJOIN_ERR_CUDA;
    }
    if ((unsigned int)(ctx->h_ctrl[1] & 0xffffffffu) != 0) return SIMJOIN_ERR_TIMEOUT;
    *count = ctx->h_ctrl[0];
    float a = 0.f, b = 0.f;
    if (cudaEventElapsedTime(&a, ctx->ev[0], ctx->ev[1]) == cudaSuccess && cudaEventElapsedTime(&b, ctx->ev[1], ctx->ev[2]) == cudaSuccess) {
        ctx->prepass_ms = a;       // hashing
        ctx->join_ms = b;          // L x (regroup + bucketed join)
        ctx->have_timing = true;
    }
    return *count > capacity ? SIMJOIN_ERR_CAPACITY : SIMJOIN_OK;
}

simjoin_status check_lsh_args(int32_t L, int32_t L_low, int32_t k, simjoin_lsh_family family = SIMJOIN_LSH_BITS) {
    if (family != SIMJOIN_LSH_BITS && family != SIMJOIN_LSH_HYPERPLANES && family != SIMJOIN_LSH_BITS_IID) return SIMJOIN_ERR_ARG;
    if (L < 0 || L_low < 0 || L + L_low < 1 || L + L_low > LSH_MAX_REPS || k < 0 || (L_low > 0 && k < 1)) return SIMJOIN_ERR_ARG;
    if (k > LSH_MAX_BITS) return SIMJOIN_ERR_UNSUPPORTED;
    return SIMJOIN_OK;
}

simjoin_status check_hamming_args(const simjoin_ctx *ctx, const void *P_bits, int64_t n, const void *Q_bits, int64_t m, int32_t d,
                                  double r, const int32_t *out_pairs, uint64_t capacity, const uint64_t *count) {
    if (!ctx || !count || !P_bits || !Q_bits) return SIMJOIN_ERR_ARG;
    if (ctx->dtype != SIMJOIN_I8) return SIMJOIN_ERR_UNSUPPORTED;
    if (n < 0 || m < 0 || n >= SIMJOIN_MAX_ROWS || m >= SIMJOIN_MAX_ROWS || d <= 0) return SIMJOIN_ERR_ARG;
    if (std::isnan(r) || r < 0) return SIMJOIN_ERR_ARG;
    if (!out_pairs && capacity > 0) return SIMJOIN_ERR_ARG;
    if (d % 128 != 0 || d > SIMJOIN_MAX_ROW_BYTES) return SIMJOIN_ERR_UNSUPPORTED;    // 16-byte packed rows
    if ((reinterpret_cast<uintptr_t>(P_bits) & 15u) || (reinterpret_cast<uintptr_t>(Q_bits) & 15u)) return SIMJOIN_ERR_UNSUPPORTED;
    if (n + ctx->ioff >= SIMJOIN_MAX_ROWS || m + ctx->joff >= SIMJOIN_MAX_ROWS) return SIMJOIN_ERR_ARG;
    return SIMJOIN_OK;
}

// Operand transform of the Hamming joins: bits -> +-1 int8 rows in the context's staging buffers.  The device must be
// current.  Leaves *count = 0.
simjoin_status hamming_unpack(simjoin_ctx *ctx, const void *P_bits, int64_t n, const void *Q_bits, int64_t m, int32_t d,
                              const int32_t *out_pairs, uint64_t capacity, uint64_t *count) {
    if ((n > 0 && !is_device_ptr(P_bits, ctx->device)) || (m > 0 && !is_device_ptr(Q_bits, ctx->device))) return SIMJOIN_ERR_ARG;
    if (capacity > 0 && !is_device_ptr(out_pairs, ctx->device)) return SIMJOIN_ERR_ARG;
    if (capacity > 0 && (reinterpret_cast<uintptr_t>(out_pairs) & 7u) != 0) return SIMJOIN_ERR_UNSUPPORTED;
    *count = 0;
    if (n == 0 || m == 0) return SIMJOIN_OK;
    const size_t pb = (size_t)n * d, qb = (size_t)m * d;
    if (!grow(ctx->stage_p, pb) || !grow(ctx->stage_q, qb)) return SIMJOIN_ERR_CUDA;
    cudaStream_t s = ctx->stream;
    const long long ph = (long long)n * d / 16, qh = (long long)m * d / 16;      // 16-bit groups
    unpack_bits_pm1_kernel<<<(unsigned)((ph + 255) / 256), 256, 0, s>>>(reinterpret_cast<const uint16_t *>(P_bits), ph,
                                                                         reinterpret_cast<uint4 *>(ctx->stage_p.ptr));
    unpack_bits_pm1_kernel<<<(unsigned)((qh + 255) / 256), 256, 0, s>>>(reinterpret_cast<const uint16_t *>(Q_bits), qh,
                                                                         reinterpret_cast<uint4 *>(ctx->stage_q.ptr));
    return cudaGetLastError() == cudaSuccess ? SIMJOIN_OK : SIMJOIN_ERR_CUDA;
}

// The JL transform (Section 3) of n rows; row r of the result starts at out + r * out_ld (out_ld >= k, a multiple of 8).
simjoin_status jl_device(simjoin_ctx *ctx, const void *X, int64_t n, int32_t d, int32_t k, uint64_t seed, void *out, int64_t out_ld) {
    if (!ctx || !X || !out || n < 0 || d <= 0 || k <= 0) return SIMJOIN_ERR_ARG;
    if (ctx->dtype != SIMJOIN_BF16) return SIMJOIN_ERR_UNSUPPORTED;
    if (d % k != 0) return SIMJOIN_ERR_ARG;
    int levels = 0;
    for (int q = d / k; q > 1; q /= 2, ++levels)
        if (q % 2 != 0) return SIMJOIN_ERR_ARG;                       // zeta = 2: d / k must be a power of two
    if (levels < 1) return SIMJOIN_ERR_ARG;
    if (k % 8 != 0) return SIMJOIN_ERR_UNSUPPORTED;                   // 16-byte rows at every level
    const int c_max = levels == 1 ? 2 * k : 2 * (levels - 1) * k;     // widest block: the last level's
    if ((size_t)c_max * 2 > SIMJOIN_MAX_ROW_BYTES || (size_t)d * 2 > SIMJOIN_MAX_ROW_BYTES) return SIMJOIN_ERR_UNSUPPORTED;
    if (n * (int64_t)(d / (2 * k)) >= SIMJOIN_MAX_ROWS) return SIMJOIN_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(X) & 15u) || (reinterpret_cast<uintptr_t>(out) & 15u)) return SIMJOIN_ERR_UNSUPPORTED;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SIMJOIN_ERR_CUDA;
    ctx->have_timing = false;
    if (n == 0) return SIMJOIN_OK;
    if (!is_device_ptr(X, ctx->device) || !is_device_ptr(out, ctx->device)) return SIMJOIN_ERR_ARG;
    // ping-pong level outputs (at most d/2 coordinates per point) and the largest level matrix
    size_t a_elems = 0, mid_elems = 0;
    for (int i = 1; i <= levels; ++i) {
        const size_t ki = i < levels ? (size_t)i * k : (size_t)k, ci = i == 1 ? (size_t)2 * k : (size_t)2 * (i - 1) * k;
        const size_t ri = (size_t)1 << (levels - i);
        if (ki * ci > a_elems) a_elems = ki * ci;
        if (i < levels && ri * ki > mid_elems) mid_elems = ri * ki;
    }
    if (!grow(ctx->jl_a, a_elems * 2) || (levels > 1 && (!grow(ctx->jl_buf[0], (size_t)n * mid_elems * 2) ||
                                                          (levels > 2 && !grow(ctx->jl_buf[1], (size_t)n * mid_elems * 2)))))
        return SIMJOIN_ERR_CUDA;
    cudaStream_t s = ctx->stream;
    ctx->ctrl_clean = -1;                         // this call uses the first control block and leaves it dirty
    if (cudaMemsetAsync(ctx->d_ctrl, 0, 64, s) != cudaSuccess) return SIMJOIN_ERR_CUDA;
    cudaEventRecord(ctx->ev[0], s);
    cudaEventRecord(ctx->ev[1], s);
    const void *src = X;
    for (int i = 1; i <= levels; ++i) {
        const int ki = i < levels ? i * k : k, ci = i == 1 ? 2 * k : 2 * (i - 1) * k;
        const int64_t rows = n * ((int64_t)1 << (levels - i));        // n * r_i blocks of c_i coordinates
        void *dst = i == levels ? out : ctx->jl_buf[(i - 1) & 1].ptr;
        jl_sign_matrix_kernel<<<(unsigned)(((long long)ki * ci + 255) / 256), 256, 0, s>>>(seed, i, ki, ci,
                                                                                         reinterpret_cast<uint16_t *>(ctx->jl_a.ptr));
        if (cudaGetLastError() != cudaSuccess) return SIMJOIN_ERR_CUDA;
        // the tile kernel with the level matrix as the resident operand and the blocks as the streamed one
        JoinParams jp;
        size_t smem = 0;
        if (!tile_geometry(ctx, ki, rows, ci * 2, 2, jp, smem)) return SIMJOIN_ERR_UNSUPPORTED;
        // a level matrix of at most 128 rows and two chunks: 256 streamed rows per tile, 32 KiB ring stages
        const bool wideq = ki <= TILE_M && jp.kc <= 2;
        const int tn = wideq ? LONG_TN : TILE_N;
        if (wideq) {
            const int p_bytes = P_BUFS * jp.kc * A_CHUNK_BYTES;
            int nstages = (ctx->max_smem_optin - 1024 - CTRL_BYTES - STAGING_BYTES - p_bytes) / LONG_Q_CHUNK_BYTES;
            if (nstages > MAX_STAGES) nstages = MAX_STAGES;
            jp.nstages = nstages;
            jp.epi_release = nstages >= 2 * jp.kc ? 1 : 0;
            smem = 1024 + (size_t)p_bytes + (size_t)nstages * LONG_Q_CHUNK_BYTES + STAGING_BYTES + CTRL_BYTES;
        }
        jp.PB = (ki + P_ROWS - 1) / P_ROWS;
        jp.QT = (int)((rows + tn - 1) / tn);
        jp.qpanel = jp.QT;                 // the blocks are read once: no L2 panels, one long sweep per CTA
        jp.counter = ctx->d_ctrl;
        jp.status = reinterpret_cast<unsigned int *>(ctx->d_ctrl + 1);
        jp.store_out = reinterpret_cast<uint16_t *>(dst);
        jp.store_ld = i == levels ? out_ld : ki;
        jp.store_scale = (float)(1.0 / std::sqrt((double)ki));
        CUtensorMap mapA, mapX;
        if (!encode_rows_map(ctx, &mapA, ctx->jl_a.ptr, ki, ci, P_ROWS) || !encode_rows_map(ctx, &mapX, src, rows, ci, tn))
            return SIMJOIN_ERR_CUDA;
        const cudaError_t le = wideq ? launch_store_wideq(ctx, mapA, mapX, jp, ctx->num_sms, smem)
                                     : launch_join<DT_BF16, KIND_STORE>(ctx, mapA, mapX, jp, ctx->num_sms, smem);
        if (le != cudaSuccess) return SIMJOIN_ERR_CUDA;
        src = dst;
    }
    cudaEventRecord(ctx->ev[2], s);
    if (cudaMemcpyAsync(ctx->h_ctrl, ctx->d_ctrl, 16, cudaMemcpyDeviceToHost, s) != cudaSuccess) return SIMJOIN_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) {
        cudaGetLastError();
        return SIMJOIN_ERR_CUDA;
    }
    if ((unsigned int)(ctx->h_ctrl[1] & 0xffffffffu) != 0) return SIMJOIN_ERR_TIMEOUT;
    float b = 0.f;
    if (cudaEventElapsedTime(&b, ctx->ev[1], ctx->ev[2]) == cudaSuccess) {
        ctx->prepass_ms = 0.f;
        ctx->join_ms = b;          // all levels
        ctx->have_timing = true;
    }
    return SIMJOIN_OK;
}

// Keep the listed pairs whose rows pass the predicate; the list is compacted in place (order unspecified).
simjoin_status filter_device(simjoin_ctx *ctx, const void *P, int64_t n, const void *Q, int64_t m, int32_t d, simjoin_kind kind,
                             double threshold, int32_t *pairs, uint64_t count_in, uint64_t *count_out) {
    *count_out = 0;
    if (count_in == 0) return SIMJOIN_OK;
    const bool i8 = ctx->dtype == SIMJOIN_I8;
    const int g = (int)((size_t)d * elem_size(ctx->dtype) / 16);
    if (!grow(ctx->filter_out, (size_t)count_in * 8)) return SIMJOIN_ERR_CUDA;
    JoinParams jp;
    std::memset(&jp, 0, sizeof jp);
    set_thresholds(jp, i8, kind, threshold);
    cudaStream_t s = ctx->stream;
    ctx->ctrl_clean = -1;                         // this call uses the first control block and leaves it dirty
    if (cudaMemsetAsync(ctx->d_ctrl, 0, 64, s) != cudaSuccess) return SIMJOIN_ERR_CUDA;
    // G lanes per pair (the power of two covering the row's 16-byte words), at most 16 blocks per SM (the warps then
    // stride over the list)
    int G = 1;
    while (G < g && G < 32) G *= 2;
    const unsigned long long want_blocks = (count_in * G + FILTER_THREADS - 1) / FILTER_THREADS;
    const unsigned long long max_blocks = (unsigned long long)ctx->num_sms * 16;
    const unsigned blocks = (unsigned)(want_blocks < max_blocks ? want_blocks : max_blocks);
    const uint4 *p4 = reinterpret_cast<const uint4 *>(P), *q4 = reinterpret_cast<const uint4 *>(Q);
    const int2 *in = reinterpret_cast<const int2 *>(pairs);
    int2 *out = reinterpret_cast<int2 *>(ctx->filter_out.ptr);
    unsigned int *status = reinterpret_cast<unsigned int *>(ctx->d_ctrl + 1);
#define SJ_FILTER(DT, KIND)                                                                                              \
    filter_pairs_kernel<DT, KIND><<<blocks, FILTER_THREADS, 0, s>>>(p4, n, q4, m, g, in, count_in, (int)ctx->ioff, (int)ctx->joff, \
                                                                    jp.thr_i, jp.thr_f, jp.thr_d, out, ctx->d_ctrl, status, G)
    if (i8 && kind == SIMJOIN_IP) SJ_FILTER(DT_I8, KIND_IP);
    else if (i8 && kind == SIMJOIN_COS) SJ_FILTER(DT_I8, KIND_COS);
    else if (i8) SJ_FILTER(DT_I8, KIND_L2);
    else if (kind == SIMJOIN_IP) SJ_FILTER(DT_BF16, KIND_IP);
    else if (kind == SIMJOIN_COS) SJ_FILTER(DT_BF16, KIND_COS);
    else SJ_FILTER(DT_BF16, KIND_L2);
#undef SJ_FILTER
    if (cudaGetLastError() != cudaSuccess) return SIMJOIN_ERR_CUDA;
    if (cudaMemcpyAsync(ctx->h_ctrl, ctx->d_ctrl, 16, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess) {
        cudaGetLastError();
        return SIMJOIN_ERR_CUDA;
    }
    if ((ctx->h_ctrl[1] & 0xffffffffu) != 0) return SIMJOIN_ERR_ARG;        // an index outside the point sets
    const uint64_t kept = ctx->h_ctrl[0];
    if (kept > 0 && (cudaMemcpyAsync(pairs, out, (size_t)kept * 8, cudaMemcpyDeviceToDevice, s) != cudaSuccess ||
                     cudaStreamSynchronize(s) != cudaSuccess)) {
        cudaGetLastError();
        return SIMJOIN_ERR_CUDA;
    }
    *count_out = kept;
    return SIMJOIN_OK;
}

}  // namespace

extern "C" {

simjoin_status simjoin_create(simjoin_ctx **out, simjoin_dtype dtype, int device, void *cuda_stream) {
    if (!out) return SIMJOIN_ERR_ARG;
    *out = nullptr;
    if (dtype != SIMJOIN_I8 && dtype != SIMJOIN_BF16) return SIMJOIN_ERR_ARG;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess) {
        cudaGetLastError();
        return SIMJOIN_ERR_CUDA;
    }
    if (device < 0 || device >= ndev) return SIMJOIN_ERR_ARG;
    int major = 0, sms = 0, smem = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) != cudaSuccess)
        return SIMJOIN_ERR_CUDA;
    if (major != 10) return SIMJOIN_ERR_ARCH;
    DeviceGuard guard(device);
    if (!guard.ok) return SIMJOIN_ERR_CUDA;
    simjoin_ctx *ctx = new (std::nothrow) simjoin_ctx();
    if (!ctx) return SIMJOIN_ERR_CUDA;
    ctx->dtype = dtype;
    ctx->device = device;
    ctx->stream = static_cast<cudaStream_t>(cuda_stream);
    ctx->num_sms = sms;
    ctx->max_smem_optin = smem;
    ctx->d_ctrl = nullptr;
    ctx->h_ctrl = nullptr;
    ctx->have_timing = false;
    ctx->ioff = ctx->joff = 0;
    ctx->ctrl_clean = -1;
    ctx->select_min_ops = DEFAULT_SELECT_MIN_OPS;
    ctx->kernel_timing = true;
    std::memset(ctx->attr_set, 0, sizeof ctx->attr_set);
    std::memset(ctx->attr_set_long, 0, sizeof ctx->attr_set_long);
    ctx->attr_set_wideq = false;
    std::memset(ctx->attr_set_dense, 0, sizeof ctx->attr_set_dense);
    std::memset(ctx->attr_set_embed, 0, sizeof ctx->attr_set_embed);
    ctx->attr_set_sign[0] = ctx->attr_set_sign[1] = false;
    ctx->dense_mode = 2;
    ctx->last_density = -1.0;
    ctx->copy_stream = nullptr;
    for (auto &e : ctx->copy_ev) e = nullptr;
    for (auto &e : ctx->ev) e = nullptr;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    bool ok = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
              qres == cudaDriverEntryPointSuccess && fn != nullptr;
    ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);
    ok = ok && cudaMalloc(reinterpret_cast<void **>(&ctx->d_ctrl), 128) == cudaSuccess;
    ok = ok && cudaMallocHost(reinterpret_cast<void **>(&ctx->h_ctrl), 128) == cudaSuccess;
    for (auto &e : ctx->ev) ok = ok && cudaEventCreate(&e) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        simjoin_destroy(ctx);
        return SIMJOIN_ERR_CUDA;
    }
    *out = ctx;
    return SIMJOIN_OK;
}

simjoin_status simjoin_destroy(simjoin_ctx *ctx) {
    if (!ctx) return SIMJOIN_OK;
    DeviceGuard guard(ctx->device);
    release(ctx->nx);
    release(ctx->ny);
    release(ctx->qstat);
    release(ctx->stage_p);
    release(ctx->stage_q);
    release(ctx->stage_out);
    release(ctx->jl_a);
    release(ctx->jl_buf[0]);
    release(ctx->jl_buf[1]);
    release(ctx->jl_p);
    release(ctx->jl_q);
    release(ctx->filter_out);
    release(ctx->lsh_keys_p);
    release(ctx->lsh_keys_q);
    release(ctx->lsh_perm_p);
    release(ctx->lsh_perm_q);
    release(ctx->lsh_sorted_p);
    release(ctx->lsh_sorted_q);
    release(ctx->lsh_misc);
    release(ctx->lsh_planes);
    release(ctx->emb_p);
    release(ctx->emb_q);
    for (auto &e : ctx->copy_ev)
        if (e) cudaEventDestroy(e);
    if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
    if (ctx->d_ctrl) cudaFree(ctx->d_ctrl);
    if (ctx->h_ctrl) cudaFreeHost(ctx->h_ctrl);
    for (auto &e : ctx->ev)
        if (e) cudaEventDestroy(e);
    delete ctx;
    return SIMJOIN_OK;
}

simjoin_status simjoin_set_offsets(simjoin_ctx *ctx, int64_t row_offset_p, int64_t row_offset_q) {
    if (!ctx || row_offset_p < 0 || row_offset_q < 0 || row_offset_p >= SIMJOIN_MAX_ROWS || row_offset_q >= SIMJOIN_MAX_ROWS)
        return SIMJOIN_ERR_ARG;
    ctx->ioff = row_offset_p;
    ctx->joff = row_offset_q;
    return SIMJOIN_OK;
}

simjoin_status simjoin_set_option(simjoin_ctx *ctx, simjoin_option option, double value) {
    if (!ctx || std::isnan(value)) return SIMJOIN_ERR_ARG;
    switch (option) {
        case SIMJOIN_OPT_SELECT_MIN_OPS:
            if (value < 0) return SIMJOIN_ERR_ARG;
            ctx->select_min_ops = value;
            return SIMJOIN_OK;
        case SIMJOIN_OPT_DENSE_EPILOGUE:
            if (value != 0.0 && value != 1.0 && value != 2.0) return SIMJOIN_ERR_ARG;
            ctx->dense_mode = (int)value;
            return SIMJOIN_OK;
        case SIMJOIN_OPT_KERNEL_TIMING:
            if (value != 0.0 && value != 1.0) return SIMJOIN_ERR_ARG;
            ctx->kernel_timing = value != 0.0;
            return SIMJOIN_OK;
    }
    return SIMJOIN_ERR_ARG;
}

simjoin_status simjoin_run(simjoin_ctx *ctx, const void *P, int64_t n, const void *Q, int64_t m, int32_t d,
                           simjoin_kind kind, double threshold, int32_t *out_pairs, uint64_t capacity, uint64_t *count) {
    simjoin_status st = check_join_args(ctx, P, n, Q, m, d, kind, threshold, out_pairs, capacity, count);
    if (st != SIMJOIN_OK) return st;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SIMJOIN_ERR_CUDA;
    if ((n > 0 && !is_device_ptr(P, ctx->device)) || (m > 0 && !is_device_ptr(Q, ctx->device))) return SIMJOIN_ERR_ARG;
    if (capacity > 0 && !is_device_ptr(out_pairs, ctx->device)) return SIMJOIN_ERR_ARG;
    if (capacity > 0 && (reinterpret_cast<uintptr_t>(out_pairs) & 7u) != 0) return SIMJOIN_ERR_UNSUPPORTED;
    return run_device(ctx, P, n, Q, m, d, kind, threshold, out_pairs, capacity, count);
}

simjoin_status simjoin_run_host(simjoin_ctx *ctx, const void *P_host, int64_t n, const void *Q_host, int64_t m, int32_t d,
                                simjoin_kind kind, double threshold, int32_t *out_pairs_host, uint64_t capacity,
                                uint64_t *count) {
    simjoin_status st = check_join_args(ctx, P_host, n, Q_host, m, d, kind, threshold, out_pairs_host, capacity, count);
    if (st != SIMJOIN_OK) return st;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SIMJOIN_ERR_CUDA;
    if (is_device_ptr(P_host, ctx->device) || is_device_ptr(Q_host, ctx->device)) return SIMJOIN_ERR_ARG;
    if (capacity > 0 && is_device_ptr(out_pairs_host, ctx->device)) return SIMJOIN_ERR_ARG;
    *count = 0;
    if (n == 0 || m == 0) return SIMJOIN_OK;
    const size_t es = elem_size(ctx->dtype);
    const size_t pb = (size_t)n * d * es, qb = (size_t)m * d * es, ob = (size_t)capacity * 8;
    if (!grow(ctx->stage_p, pb) || !grow(ctx->stage_q, qb) || !grow(ctx->stage_out, ob ? ob : 8)) return SIMJOIN_ERR_CUDA;
    cudaStream_t s = ctx->stream;
    // A large Q goes up in slices of about 32 MiB on a second stream, and each slice is joined (a call of its own,
    // with the column offset of the slice) as soon as it has landed: the copies of the later slices hide behind
    // the joins of the earlier ones.  The result is the union of the slices' results.  A caller that provides room
    // for a large output (64 MiB of pairs and more) gets slices too, eight of them: the pairs of a slice travel back
    // to the host on the second stream while the next slice is joined.
    const size_t row_bytes = (size_t)d * es;
    int64_t slice_rows = m;
    if (qb > (64u << 20)) slice_rows = (int64_t)(((32u << 20) / row_bytes + TILE_N - 1) / TILE_N * TILE_N);
    else if (ob >= (64u << 20) && m >= 8 * 4096) slice_rows = ((m + 7) / 8 + LONG_TN - 1) / LONG_TN * LONG_TN;
    // a Q of 32 to 64 MiB: four slices (measured on 262 144 x 256 int8: 2897 -> 3179 TOPS end to end; a 16 MiB Q loses in four
    // slices, 820 -> 752, because each slice's join is then only ~0.2 ms against ~35 us of per-call overhead)
    else if (qb >= (32u << 20) && m >= 4 * 8192) slice_rows = ((m + 3) / 4 + LONG_TN - 1) / LONG_TN * LONG_TN;
    const int nslices = (int)((m + slice_rows - 1) / slice_rows);
    static_assert(sizeof(((simjoin_ctx *)nullptr)->copy_ev) / sizeof(cudaEvent_t) == MAX_HOST_SLICES + 1, "one event per slice and one more");
    if (nslices > 1 && nslices <= MAX_HOST_SLICES) {
        if (!ctx->copy_stream && cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking) != cudaSuccess) return SIMJOIN_ERR_CUDA;
        for (int q = 0; q <= nslices; ++q)
            if (!ctx->copy_ev[q] && cudaEventCreateWithFlags(&ctx->copy_ev[q], cudaEventDisableTiming) != cudaSuccess) return SIMJOIN_ERR_CUDA;
        cudaStream_t cs = ctx->copy_stream;
        // Nothing the caller passes may be in use after the call returns: an error exit waits for the copies
        // already enqueued from the caller's buffers.
        auto fail = [&](simjoin_status code) {
            cudaStreamSynchronize(cs);
            cudaGetLastError();
            return code;
        };
        // the staging buffers may still be in use by earlier work on the context's stream
        if (cudaEventRecord(ctx->copy_ev[nslices], s) != cudaSuccess || cudaStreamWaitEvent(cs, ctx->copy_ev[nslices], 0) != cudaSuccess)
            return fail(SIMJOIN_ERR_CUDA);
        if (cudaMemcpyAsync(ctx->stage_p.ptr, P_host, pb, cudaMemcpyHostToDevice, cs) != cudaSuccess) return fail(SIMJOIN_ERR_CUDA);
        for (int q = 0; q < nslices; ++q) {
            const int64_t r0 = q * slice_rows, rows = (m - r0 < slice_rows) ? m - r0 : slice_rows;
            if (cudaMemcpyAsync(static_cast<char *>(ctx->stage_q.ptr) + (size_t)r0 * row_bytes, static_cast<const char *>(Q_host) + (size_t)r0 * row_bytes,
                                (size_t)rows * row_bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess ||
                cudaEventRecord(ctx->copy_ev[q], cs) != cudaSuccess)
                return fail(SIMJOIN_ERR_CUDA);
        }
        const long long joff0 = ctx->joff;
        uint64_t total = 0;
        float pre_ms = 0.f, join_ms = 0.f;
        st = SIMJOIN_OK;
        for (int q = 0; q < nslices && (st == SIMJOIN_OK || st == SIMJOIN_ERR_CAPACITY); ++q) {
            const int64_t r0 = q * slice_rows, rows = (m - r0 < slice_rows) ? m - r0 : slice_rows;
            if (cudaStreamWaitEvent(s, ctx->copy_ev[q], 0) != cudaSuccess) { st = SIMJOIN_ERR_CUDA; break; }
            const uint64_t used = total < capacity ? total : capacity;
            uint64_t cnt = 0;
            ctx->joff = joff0 + r0;
            const simjoin_status sq = run_device(ctx, ctx->stage_p.ptr, n, static_cast<char *>(ctx->stage_q.ptr) + (size_t)r0 * row_bytes, rows, d, kind,
                                                 threshold, capacity > used ? reinterpret_cast<int32_t *>(ctx->stage_out.ptr) + 2 * used : nullptr,
                                                 capacity - used, &cnt);
            ctx->joff = joff0;
            total += cnt;
            if (sq != SIMJOIN_OK) st = sq;
            if (ctx->have_timing) { pre_ms += ctx->prepass_ms; join_ms += ctx->join_ms; }
            // the slice's join has finished (run_device synchronises): its pairs go home behind the next slice's join
            const uint64_t now = total < capacity ? total : capacity;
            if ((sq == SIMJOIN_OK || sq == SIMJOIN_ERR_CAPACITY) && now > used &&
                cudaMemcpyAsync(out_pairs_host + 2 * used, reinterpret_cast<int32_t *>(ctx->stage_out.ptr) + 2 * used,
                                (size_t)(now - used) * 8, cudaMemcpyDeviceToHost, cs) != cudaSuccess)
                st = SIMJOIN_ERR_CUDA;
        }
        if (cudaStreamSynchronize(cs) != cudaSuccess) {
            cudaGetLastError();
            return SIMJOIN_ERR_CUDA;
        }
        if (st != SIMJOIN_OK && st != SIMJOIN_ERR_CAPACITY) return st;
        ctx->prepass_ms = pre_ms;
        ctx->join_ms = join_ms;
        *count = total;
        return total > capacity ? SIMJOIN_ERR_CAPACITY : SIMJOIN_OK;
    } else {
        if (cudaMemcpyAsync(ctx->stage_p.ptr, P_host, pb, cudaMemcpyHostToDevice, s) != cudaSuccess ||
            cudaMemcpyAsync(ctx->stage_q.ptr, Q_host, qb, cudaMemcpyHostToDevice, s) != cudaSuccess)
            return SIMJOIN_ERR_CUDA;
        st = run_device(ctx, ctx->stage_p.ptr, n, ctx->stage_q.ptr, m, d, kind, threshold,
                        capacity ? reinterpret_cast<int32_t *>(ctx->stage_out.ptr) : nullptr, capacity, count);
        if (st != SIMJOIN_OK && st != SIMJOIN_ERR_CAPACITY) return st;
    }
    const uint64_t wrote = *count < capacity ? *count : capacity;
    if (wrote > 0) {
        if (cudaMemcpyAsync(out_pairs_host, ctx->stage_out.ptr, (size_t)wrote * 8, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
            cudaStreamSynchronize(s) != cudaSuccess) {
            cudaGetLastError();
            return SIMJOIN_ERR_CUDA;
        }
    }
    return st;
}

simjoin_status simjoin_run_hamming(simjoin_ctx *ctx, const void *P_bits, int64_t n, const void *Q_bits, int64_t m, int32_t d,
                                   double r, int32_t *out_pairs, uint64_t capacity, uint64_t *count) {
    simjoin_status st = check_hamming_args(ctx, P_bits, n, Q_bits, m, d, r, out_pairs, capacity, count);
    if (st != SIMJOIN_OK) return st;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SIMJOIN_ERR_CUDA;
    st = hamming_unpack(ctx, P_bits, n, Q_bits, m, d, out_pairs, capacity, count);
    if (st != SIMJOIN_OK || n == 0 || m == 0) return st;
    // Hamming <= r  <=>  Hamming <= floor(r)  <=>  d - 2*Hamming >= d - 2*floor(r)
    const double t = (double)d - 2.0 * std::floor(r);
    return run_device(ctx, ctx->stage_p.ptr, n, ctx->stage_q.ptr, m, d, SIMJOIN_IP, t, out_pairs, capacity, count);
}

simjoin_status simjoin_run_lsh(simjoin_ctx *ctx, const void *P, int64_t n, const void *Q, int64_t m, int32_t d,
                               simjoin_kind kind, double threshold, simjoin_lsh_family family, int32_t L, int32_t L_low, int32_t k,
                               uint64_t seed, int32_t *out_pairs, uint64_t capacity, uint64_t *count) {
    simjoin_status st = check_join_args(ctx, P, n, Q, m, d, kind, threshold, out_pairs, capacity, count);
    if (st != SIMJOIN_OK) return st;
    st = check_lsh_args(L, L_low, k, family);
    if (st != SIMJOIN_OK) return st;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SIMJOIN_ERR_CUDA;
    if ((n > 0 && !is_device_ptr(P, ctx->device)) || (m > 0 && !is_device_ptr(Q, ctx->device))) return SIMJOIN_ERR_ARG;
    if (capacity > 0 && !is_device_ptr(out_pairs, ctx->device)) return SIMJOIN_ERR_ARG;
    if (capacity > 0 && (reinterpret_cast<uintptr_t>(out_pairs) & 7u) != 0) return SIMJOIN_ERR_UNSUPPORTED;
    return lsh_device(ctx, P, n, Q, m, d, kind, threshold, family, L, L_low, k, seed, out_pairs, capacity, count);
}

simjoin_status simjoin_run_hamming_lsh(simjoin_ctx *ctx, const void *P_bits, int64_t n, const void *Q_bits, int64_t m, int32_t d,
                                       double r, int32_t L, int32_t L_low, int32_t k, uint64_t seed, int32_t *out_pairs,
                                       uint64_t capacity, uint64_t *count) {
    simjoin_status st = check_hamming_args(ctx, P_bits, n, Q_bits, m, d, r, out_pairs, capacity, count);
    if (st != SIMJOIN_OK) return st;
    st = check_lsh_args(L, L_low, k);
    if (st != SIMJOIN_OK) return st;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SIMJOIN_ERR_CUDA;
    st = hamming_unpack(ctx, P_bits, n, Q_bits, m, d, out_pairs, capacity, count);
    if (st != SIMJOIN_OK || n == 0 || m == 0) return st;
    const double t = (double)d - 2.0 * std::floor(r);
    return lsh_device(ctx, ctx->stage_p.ptr, n, ctx->stage_q.ptr, m, d, SIMJOIN_IP, t, SIMJOIN_LSH_BITS, L, L_low, k, seed, out_pairs, capacity, count);
}

simjoin_status simjoin_jl_transform(simjoin_ctx *ctx, const void *X, int64_t n, int32_t d, int32_t k, uint64_t seed, void *out) {
    return jl_device(ctx, X, n, d, k, seed, out, k);
}

simjoin_status simjoin_filter_pairs(simjoin_ctx *ctx, const void *P, int64_t n, const void *Q, int64_t m, int32_t d,
                                    simjoin_kind kind, double threshold, int32_t *pairs, uint64_t count_in, uint64_t *count_out) {
    if (!count_out) return SIMJOIN_ERR_ARG;
    simjoin_status st = check_join_args(ctx, P, n, Q, m, d, kind, threshold, pairs, count_in, count_out);
    if (st != SIMJOIN_OK) return st;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SIMJOIN_ERR_CUDA;
    *count_out = 0;
    if (count_in == 0) return SIMJOIN_OK;
    if (n == 0 || m == 0) return SIMJOIN_ERR_ARG;                        // a listed pair cannot exist
    if (!is_device_ptr(P, ctx->device) || !is_device_ptr(Q, ctx->device) || !is_device_ptr(pairs, ctx->device)) return SIMJOIN_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(pairs) & 7u) != 0) return SIMJOIN_ERR_UNSUPPORTED;
    ctx->have_timing = false;
    return filter_device(ctx, P, n, Q, m, d, kind, threshold, pairs, count_in, count_out);
}

simjoin_status simjoin_run_jl_l2(simjoin_ctx *ctx, const void *P, int64_t n, const void *Q, int64_t m, int32_t d, double r,
                                 int32_t k, uint64_t seed, double slack, int32_t *out_pairs, uint64_t capacity, uint64_t *count) {
    simjoin_status st = check_join_args(ctx, P, n, Q, m, d, SIMJOIN_L2, r, out_pairs, capacity, count);
    if (st != SIMJOIN_OK) return st;
    if (ctx->dtype != SIMJOIN_BF16) return SIMJOIN_ERR_UNSUPPORTED;
    if (std::isnan(slack) || slack < 0 || std::isinf(slack)) return SIMJOIN_ERR_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SIMJOIN_ERR_CUDA;
    if ((n > 0 && !is_device_ptr(P, ctx->device)) || (m > 0 && !is_device_ptr(Q, ctx->device))) return SIMJOIN_ERR_ARG;
    if (capacity > 0 && !is_device_ptr(out_pairs, ctx->device)) return SIMJOIN_ERR_ARG;
    if (capacity > 0 && (reinterpret_cast<uintptr_t>(out_pairs) & 7u) != 0) return SIMJOIN_ERR_UNSUPPORTED;
    *count = 0;
    if (n == 0 || m == 0) return simjoin_jl_transform(ctx, P, 0, d, k, seed, const_cast<void *>(P));   // shape rules only
    // The reduced points are joined as they are, by the Euclidean kind.  Section 4's squared-L2 embedding -- 8 appended
    // coordinates (x, -|x|^2/2, 1) . (y, 1, -|y|^2/2) = -|x - y|^2 / 2, an inner-product join with a constant threshold
    // and an exact row-maximum filter -- was measured and dropped: the 16 extra bytes per row open a second (third)
    // chunk with a short tail, and the reduced join took 15.9 ms instead of 11.8 (k = 128; 3.35 against 3.2-3.3 at k = 64).
    if (!grow(ctx->jl_p, (size_t)n * k * 2) || !grow(ctx->jl_q, (size_t)m * k * 2)) return SIMJOIN_ERR_CUDA;
    cudaStream_t s = ctx->stream;
    // the same M for both sets: |M x - M y| = |M (x - y)| is within a factor 1 +- eps of |x - y|
    st = jl_device(ctx, P, n, d, k, seed, ctx->jl_p.ptr, k);
    if (st != SIMJOIN_OK) return st;
    float jl_ms = ctx->have_timing ? ctx->join_ms : 0.f;
    st = jl_device(ctx, Q, m, d, k, seed, ctx->jl_q.ptr, k);
    if (st != SIMJOIN_OK) return st;
    jl_ms += ctx->have_timing ? ctx->join_ms : 0.f;
    // Order the reduced rows of Q by norm (counting sort on 12 bits of the norm): the join's per-tile bound is built
    // from the smallest |y|^2 of each 256-row block, and the reduced norms spread (measured at k = 64: the join of
    // the unordered rows 2.46 ms, 7 % of the warp blocks entering the exact test for nothing).
    const int nb = LSH_MAX_BUCKETS;
    const int g = k * 2 / 16;
    if (!grow(ctx->nx, (size_t)m * 4) || !grow(ctx->lsh_keys_q, (size_t)m * 2) || !grow(ctx->lsh_perm_q, (size_t)m * 4) ||
        !grow(ctx->lsh_misc, (size_t)2 * nb * 4 + 16) || !grow(ctx->lsh_sorted_q, (size_t)m * k * 2))
        return SIMJOIN_ERR_CUDA;
    {
        float *ny = reinterpret_cast<float *>(ctx->nx.ptr);
        uint16_t *keys = reinterpret_cast<uint16_t *>(ctx->lsh_keys_q.ptr);
        int *perm = reinterpret_cast<int *>(ctx->lsh_perm_q.ptr);
        unsigned int *hist = reinterpret_cast<unsigned int *>(ctx->lsh_misc.ptr), *cursor = hist + nb, *range = cursor + nb;
        // running minimum starts at 0x7f7f7f7f (3.4e38, above every norm), running maximum at 0
        if (launch_norms<false>(ctx, ctx->jl_q.ptr, m, k, 0, ny, nullptr) != cudaSuccess ||
            cudaMemsetAsync(hist, 0, (size_t)nb * 4, s) != cudaSuccess ||
            cudaMemsetAsync(range, 0x7f, 4, s) != cudaSuccess || cudaMemsetAsync(range + 1, 0, 4, s) != cudaSuccess)
            return SIMJOIN_ERR_CUDA;
        const int rows_per_block = LSH_SORT_THREADS * LSH_SORT_ITEMS;
        norm_range_kernel<<<ctx->num_sms * 4, 256, 0, s>>>(ny, m, range);
        norm_keys_kernel<<<(unsigned)((m + 255) / 256), 256, 0, s>>>(ny, m, range, nb, keys);
        lsh_hist_kernel<<<(unsigned)ctx->num_sms * 4, LSH_SORT_THREADS, 0, s>>>(keys, 1, m, nb, hist);
        hist_offsets_kernel<<<1, 1024, 0, s>>>(hist, nb, cursor);
        lsh_scatter_kernel<<<(unsigned)((m + rows_per_block - 1) / rows_per_block), LSH_SORT_THREADS, 0, s>>>(keys, 1, m, nb, cursor, perm);
        lsh_gather_rows_kernel<<<(unsigned)(((long long)m * g + 255) / 256), 256, 0, s>>>(
            reinterpret_cast<const uint4 *>(ctx->jl_q.ptr), perm, m, g, reinterpret_cast<uint4 *>(ctx->lsh_sorted_q.ptr));
        if (cudaGetLastError() != cudaSuccess) return SIMJOIN_ERR_CUDA;
    }
    // candidates: the join of the reduced points with the radius widened by the slack
    uint64_t cand = 0;
    st = run_device(ctx, ctx->jl_p.ptr, n, ctx->lsh_sorted_q.ptr, m, k, SIMJOIN_L2, r * (1.0 + slack), out_pairs, capacity, &cand);
    const float join_ms = ctx->have_timing ? ctx->prepass_ms + ctx->join_ms : 0.f;
    if (st == SIMJOIN_ERR_CAPACITY) {
        *count = cand;                  // more candidates than room: nothing can be decided
        return st;
    }
    if (st != SIMJOIN_OK) return st;
    cudaEventRecord(ctx->ev[0], s);
    if (cand > 0) {
        remap_second_index_kernel<<<(unsigned)((cand + 255) / 256), 256, 0, s>>>(reinterpret_cast<int2 *>(out_pairs), cand,
                                                                               reinterpret_cast<const int *>(ctx->lsh_perm_q.ptr), (int)ctx->joff);
        if (cudaGetLastError() != cudaSuccess) return SIMJOIN_ERR_CUDA;
    }
    st = filter_device(ctx, P, n, Q, m, d, SIMJOIN_L2, r, out_pairs, cand, count);
    cudaEventRecord(ctx->ev[1], s);
    float f_ms = 0.f;
    if (st == SIMJOIN_OK && cudaEventSynchronize(ctx->ev[1]) == cudaSuccess && cudaEventElapsedTime(&f_ms, ctx->ev[0], ctx->ev[1]) == cudaSuccess) {
        ctx->prepass_ms = jl_ms;
        ctx->join_ms = join_ms + f_ms;
        ctx->have_timing = true;
    }
    return st;
}

simjoin_status simjoin_row_norms(simjoin_ctx *ctx, const void *X, int64_t rows, int32_t d, void *out) {
    if (!ctx || !out) return SIMJOIN_ERR_ARG;
    simjoin_status st = check_matrix_args(ctx, X, rows, d);
    if (st != SIMJOIN_OK) return st;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SIMJOIN_ERR_CUDA;
    if (rows == 0) return SIMJOIN_OK;
    if (!is_device_ptr(X, ctx->device) || !is_device_ptr(out, ctx->device)) return SIMJOIN_ERR_ARG;
    const cudaError_t e = ctx->dtype == SIMJOIN_I8 ? launch_norms<true>(ctx, X, rows, d, 0, out, nullptr)
                                                   : launch_norms<false>(ctx, X, rows, d, 0, out, nullptr);
    if (e != cudaSuccess || cudaStreamSynchronize(ctx->stream) != cudaSuccess) {
        cudaGetLastError();
        return SIMJOIN_ERR_CUDA;
    }
    return SIMJOIN_OK;
}

simjoin_status simjoin_selftest_wait_timeout(simjoin_ctx *ctx) {
    if (!ctx) return SIMJOIN_ERR_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SIMJOIN_ERR_CUDA;
    cudaStream_t s = ctx->stream;
    ctx->ctrl_clean = -1;                         // this call uses the first control block and leaves it dirty
    if (cudaMemsetAsync(ctx->d_ctrl, 0, 64, s) != cudaSuccess) return SIMJOIN_ERR_CUDA;
    wait_timeout_selftest_kernel<<<1, 32, 0, s>>>(reinterpret_cast<unsigned int *>(ctx->d_ctrl + 1), 2000000LL);   // ~1 ms
    if (cudaGetLastError() != cudaSuccess ||
        cudaMemcpyAsync(ctx->h_ctrl, ctx->d_ctrl, 16, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess) {
        cudaGetLastError();
        return SIMJOIN_ERR_CUDA;
    }
    const unsigned int kstatus = (unsigned int)(ctx->h_ctrl[1] & 0xffffffffu);
    return kstatus == (0x80000000u | 0x7fu) ? SIMJOIN_ERR_TIMEOUT : SIMJOIN_ERR_CUDA;
}

simjoin_status simjoin_last_kernel_ms(simjoin_ctx *ctx, float *prepass_ms, float *join_ms) {
    if (!ctx || !ctx->have_timing) return SIMJOIN_ERR_ARG;
    if (prepass_ms) *prepass_ms = ctx->prepass_ms;
    if (join_ms) *join_ms = ctx->join_ms;
    return SIMJOIN_OK;
}

// ------------------------------------------------------------------------------------
// Allocation-free variant (no counterpart in the paper).  All scratch of the norm pre-pass
// and the join kernel lives in one file-scope device array; its device address is looked up
// once per device with cudaGetSymbolAddress (the array's name is only a host-side stand-in
// and must never be handed to a kernel directly).
namespace {

constexpr size_t NA_ROWS = SIMJOIN_NOALLOC_MAX_ROWS;
constexpr size_t NA_OFF_CTRL = 0;                                    // 64 B counter / status block
constexpr size_t NA_OFF_NX = 256;                                    // NA_ROWS x 4 B
constexpr size_t NA_OFF_NY = NA_OFF_NX + NA_ROWS * 4;                // NA_ROWS x 4 B
constexpr size_t NA_OFF_QSTAT = NA_OFF_NY + NA_ROWS * 4;             // (NA_ROWS / 256) x 8 B
constexpr size_t NA_BYTES = NA_OFF_QSTAT + (NA_ROWS / NORM_TILE_ROWS) * 8 + 256;

static __device__ __align__(256) unsigned char g_noalloc_scratch[NA_BYTES];

constexpr int NA_MAX_DEVICES = 64;
struct NoAllocDevice {
    bool ready;
    unsigned char *scratch;   // device address of g_noalloc_scratch on this device
    // A context that owns nothing (no buffers, no events, no second stream): it carries the device's limits and the
    // "kernel attribute already set" flags from call to call; dtype and stream are filled in per call.
    simjoin_ctx ctx;
};
NoAllocDevice g_na_dev[NA_MAX_DEVICES];

// Once per device, with that device current.
simjoin_status noalloc_setup(int device) {
    NoAllocDevice &nd = g_na_dev[device];
    if (nd.ready) return SIMJOIN_OK;
    int major = 0, sms = 0, smem = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) != cudaSuccess) {
        cudaGetLastError();
        return SIMJOIN_ERR_CUDA;
    }
    if (major != 10) return SIMJOIN_ERR_ARCH;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn) {
        cudaGetLastError();
        return SIMJOIN_ERR_CUDA;
    }
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) {
        cudaGetLastError();
        return SIMJOIN_ERR_CUDA;
    }
    nd.scratch = static_cast<unsigned char *>(ptr);
    nd.ctx = simjoin_ctx{};
    nd.ctx.device = device;
    nd.ctx.num_sms = sms;
    nd.ctx.max_smem_optin = smem;
    nd.ctx.encode = reinterpret_cast<EncodeTiledFn>(fn);
    nd.ready = true;
    return SIMJOIN_OK;
}

}  // namespace

simjoin_status simjoin_run_noalloc(int device, void *cuda_stream, simjoin_dtype dtype, const void *P, int64_t n,
                                   const void *Q, int64_t m, int32_t d, simjoin_kind kind, double threshold,
                                   int32_t *out_pairs, uint64_t capacity, uint64_t *count) {
    if (dtype != SIMJOIN_I8 && dtype != SIMJOIN_BF16) return SIMJOIN_ERR_ARG;
    if (device < 0 || device >= NA_MAX_DEVICES) return SIMJOIN_ERR_ARG;
    {
        simjoin_ctx probe{};       // argument checks only need the element type (offsets are zero)
        probe.dtype = dtype;
        const simjoin_status st = check_join_args(&probe, P, n, Q, m, d, kind, threshold, out_pairs, capacity, count);
        if (st != SIMJOIN_OK) return st;
    }
    if ((uint64_t)n > NA_ROWS || (uint64_t)m > NA_ROWS) return SIMJOIN_ERR_UNSUPPORTED;   // beyond the static scratch
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess) {
        cudaGetLastError();
        return SIMJOIN_ERR_CUDA;
    }
    if (device >= ndev) return SIMJOIN_ERR_ARG;
    DeviceGuard guard(device);
    if (!guard.ok) return SIMJOIN_ERR_CUDA;
    simjoin_status st = noalloc_setup(device);
    if (st != SIMJOIN_OK) return st;
    NoAllocDevice &nd = g_na_dev[device];
    if ((n > 0 && !is_device_ptr(P, device)) || (m > 0 && !is_device_ptr(Q, device))) return SIMJOIN_ERR_ARG;
    if (capacity > 0 && !is_device_ptr(out_pairs, device)) return SIMJOIN_ERR_ARG;
    if (capacity > 0 && (reinterpret_cast<uintptr_t>(out_pairs) & 7u) != 0) return SIMJOIN_ERR_UNSUPPORTED;
    nd.ctx.dtype = dtype;
    nd.ctx.stream = static_cast<cudaStream_t>(cuda_stream);
    // The same code path as simjoin_run from here on -- same geometry choice, pre-passes and kernel instantiations --
    // with its working memory in the fixed array (n, m <= NA_ROWS: whole tiles of Q never pass the end of ny) and the
    // counter read back into two words on this stack.
    unsigned long long host_ctrl[2] = {0, 0};
    const JoinScratch scr{nd.scratch + NA_OFF_NX, nd.scratch + NA_OFF_NY, nd.scratch + NA_OFF_QSTAT,
                          reinterpret_cast<unsigned long long *>(nd.scratch + NA_OFF_CTRL), host_ctrl, false};
    return run_device(&nd.ctx, P, n, Q, m, d, kind, threshold, out_pairs, capacity, count, &scr);
}

const char *simjoin_strerror(simjoin_status status) {
    switch (status) {
        case SIMJOIN_OK: return "ok";
        case SIMJOIN_ERR_ARG: return "invalid argument";
        case SIMJOIN_ERR_UNSUPPORTED: return "unsupported shape, alignment or dtype/kind combination";
        case SIMJOIN_ERR_CAPACITY: return "more passing pairs than the output capacity";
        case SIMJOIN_ERR_CUDA: return "a CUDA call failed";
        case SIMJOIN_ERR_TIMEOUT: return "a bounded wait inside the join kernel expired";
        case SIMJOIN_ERR_ARCH: return "device is not compute capability 10.x";
    }
    return "unknown status";
}

}  // extern "C"
