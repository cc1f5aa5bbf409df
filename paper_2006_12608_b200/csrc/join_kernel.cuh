// The fused similarity-join kernel for sm_100a.
//
// Section 4 of the paper reduces the join to the product F_P * G_Q^T and Theorem 1
// decomposes that product into small dense tile products.  Here one tile product is a
// 256 x 128 block of scores: 256 rows of P (two 128-row MMA blocks) against 128 rows of Q over
// all d coordinates, computed by tcgen05.mma from 128-byte-swizzled shared-memory tiles that TMA fills, with
// the accumulator in tensor memory.  The rest of the ip-distance (row norms, Section 4's
// squared-L2 and cosine forms) and the threshold are applied to the accumulator in
// registers and passing (i, j) are compacted straight into the output list.
//
// CTA layout (384 threads, one CTA per SM, persistent):
//   warp 0      TMA producer (one elected lane): P tile (resident while its Q sweep lasts) + Q chunk ring
//   warps 1, 3  MMA issuers: warp 1 even tiles -> accumulator 0, warp 3 odd tiles -> accumulator 1
//   warp 2      TMEM allocation / release
//   warps 4-11  epilogue: warp w reads TMEM lanes 32*(w%4).. of P block (w-4)/4; row max vs a
//               per-tile bound, then 16-column group maxima, then the exact test; passing pairs go
//               through a per-warp shared-memory staging buffer to the output list
// Dense outputs (bf16, rows of one or two chunks) run with 16 epilogue warps (EW = 16, 640 threads): two warps share a
// block of rows and split its 128 columns -- or, for the sign test on transformed operands, take alternate tiles.
// Every mbarrier wait is bounded; on expiry the CTA raises a status word and drains.
#pragma once
#include <cuda_bf16.h>

#include <type_traits>

#include "ptx_sm100.cuh"

namespace sj {

constexpr int DT_I8 = 0, DT_BF16 = 1;
constexpr int KIND_IP = 0, KIND_COS = 1, KIND_L2 = 2;
// KIND_STORE (bf16): no predicate -- the scaled score tile itself is written out, transposed, as bf16:
// out[j * store_ld + i] = bf16(store_scale * <P_i, Q_j>).  This is the dense product Q * P^T with P the
// small, resident operand: one level of the JL transform of Section 3.
constexpr int KIND_STORE = 3;
// KIND_SIGN (both element types): no predicate either -- the signs of the score tile are written out as hash keys.
// P holds hyperplanes, 16 rows per repetition of the LSH join (unused rows are zero), Q the points: the 32 signs
// [<P_i, Q_j> > 0] of the rows 32 w .. 32 w + 31 form word w of point j's key record, i.e. the 16-bit keys of
// repetitions 2 w and 2 w + 1:  key_out[j * key_ld + w].  This is the random-hyperplane LSH of Section 4's LSH join
// computed as the dense product it is; int8 projections are exact integers.
constexpr int KIND_SIGN = 4;

// One tile is 256 rows of P (two 128-row MMA blocks, both resident in shared memory) against 128 rows of Q.
// Every Q chunk that arrives is multiplied with both P blocks, so a tile needs half the L2 -> shared-memory
// traffic of a 128 x 256 tile for the same work.  Measured on B200 under the 1000 W cap with a skeleton of
// this pipeline: streaming 32 KiB per 512 tensor cycles costs 16 % of the SM clock (1400 vs 1630 MHz with
// the traffic switched off); at 16 KiB it costs 7 % (1505 MHz) -- the kernel is power-bound, so energy per
// tile, not cycles per tile, sets its speed.  (tcgen05.mma with N = 128 issues in 69 cycles against 64
// ideal: the tile takes 552 cycles instead of 549.)
constexpr int TILE_M = 128;                       // rows of P per MMA block (TMEM lanes)
constexpr int P_SUB = 2;                          // MMA blocks per P tile
constexpr int P_ROWS = P_SUB * TILE_M;            // rows of P per tile
constexpr int TILE_N = 128;                       // rows of Q per tile
constexpr int QSTAT_ROWS = 256;                   // rows of Q behind one (min, max) entry of the per-tile bound: two tiles
constexpr int ACC_COLS = P_SUB * TILE_N;          // TMEM columns of one accumulator buffer: block s at s * TILE_N
constexpr int CHUNK_BYTES = 128;                  // K bytes per shared-memory chunk (one swizzle atom)
constexpr int A_CHUNK_BYTES = P_ROWS * CHUNK_BYTES;   // 32 KiB: one K chunk of both P blocks (block s at s * 16 KiB)
constexpr int A_SUB_BYTES = TILE_M * CHUNK_BYTES;     // 16 KiB
constexpr int B_CHUNK_BYTES = TILE_N * CHUNK_BYTES;   // 16 KiB
constexpr int MAX_STAGES = 8;
// long-row and wide-Q geometries (see join_kernel): 256 rows of Q per tile
constexpr int LONG_TN = 2 * TILE_N;                           // rows of Q per long tile
constexpr int LONG_Q_CHUNK_BYTES = LONG_TN * CHUNK_BYTES;     // 32 KiB
constexpr int LONG_STAGE_BYTES = LONG_Q_CHUNK_BYTES + A_CHUNK_BYTES;
constexpr int LONG_STAGES = 3;
constexpr int MAX_STATIONARY_CHUNKS = 4;          // P block kept resident up to 512-byte rows
constexpr int P_BUFS = 1;                         // resident P tiles of the sweep schedule (a short bubble per Q sweep)
// Bucketed mode sweeps only a bucket's Q rows per P block (tens of tiles, not thousands): there the bubble
// matters, and the next P block is fetched while the current one is still being multiplied (rows of up to
// two chunks; longer rows would pay for the second block with ring depth).
__host__ __device__ constexpr int p_bufs(bool grouped, int kc) { return grouped && kc <= 2 ? 2 : P_BUFS; }
constexpr int EPI_WARP0 = 4;
constexpr int NUM_EPI_WARPS = 4 * P_SUB;                       // one per TMEM lane quarter and P block
constexpr int EPI_COLS = TILE_N;                               // accumulator columns per epilogue warp
constexpr int NUM_THREADS = 32 * (EPI_WARP0 + NUM_EPI_WARPS);
constexpr uint32_t TMEM_COLS = 512;
constexpr long long WAIT_LIMIT_CYCLES = 2000000000LL;  // ~1 s: far beyond any legitimate wait
constexpr int CTRL_BYTES = 256;
constexpr int WARP_STAGE_BYTES = 2048;                           // per epilogue warp: staged pairs, then the column terms
constexpr int COLTERM_BYTES = EPI_COLS * 4;                      // per-column terms of the 128 columns under test
constexpr int STAGE_PAIRS = (WARP_STAGE_BYTES - COLTERM_BYTES) / 8;   // pairs staged in shared memory per warp
constexpr int STAGING_BYTES = NUM_EPI_WARPS * WARP_STAGE_BYTES;  // 16 KiB
// The dense-output instantiations run 16 epilogue warps (EW = 16): four per TMEM lane quarter, each taking 64 of a P
// block's 128 columns, on the same 16 KiB of staging (1 KiB per warp).  A join whose every 32 x 128 block holds hits is
// bound by the dependent-issue latency of the element tests, which twice the warps hide; a sparse join is bound by the
// throughput of the row maxima and is faster with 8 warps of 128 columns (fewer, longer trees).
__host__ __device__ constexpr int epi_cols(int ew) { return TILE_N * NUM_EPI_WARPS / ew; }
__host__ __device__ constexpr int warp_stage_bytes(int ew) { return STAGING_BYTES / ew; }
__host__ __device__ constexpr int stage_pairs(int ew) { return (warp_stage_bytes(ew) - epi_cols(ew) * 4) / 8; }
__host__ __device__ constexpr int num_threads(int ew) { return 32 * (EPI_WARP0 + ew); }
static_assert(stage_pairs(NUM_EPI_WARPS) == STAGE_PAIRS && num_threads(NUM_EPI_WARPS) == NUM_THREADS, "");

struct JoinParams {
    long long n, m;          // rows of P, Q
    int kc;                  // 128-byte K chunks per row = ceil(row_bytes / 128)
    int last_ksteps;         // 32-byte MMA K steps in the last chunk (1..4)
    int elems_per_chunk;     // 128 / sizeof(element)
    int stationary;          // 1: the P block stays in shared memory for its whole Q sweep
    int nstages;             // ring depth
    int epi_release;         // 1: the epilogue hands ring stages back (one commit per tile); needs nstages >= 2*kc
    int PB, QT;              // number of 256-row P tiles, 128-row Q tiles
    int qpanel;              // Q tiles per L2-resident panel
    int wave_gq;             // > 0: two-dimensional waves, (gridDim / wave_gq) P tiles x wave_gq Q tiles at a time (very long rows)
    int thr_i;               // I8/IP: ceil(t);  I8/L2: floor(r*r); both clamped
    float thr_f;             // BF16: t (IP, COS) or r*r (L2)
    const void *nx;          // per-row term of P: int32 |x|^2 (I8/L2), fp32 |x| (COS, both element types) or |x|^2 (BF16/L2)
    const void *ny;          // same for Q
    const void *qstat;       // per 256 rows of Q (two tiles): (min, max) of ny over the valid rows
    int2 *out;               // capacity x (i, j)
    unsigned long long capacity;
    unsigned long long *counter;   // total passing pairs
    unsigned int *status;          // 0 = ok, else 0x80000000 | wait site that timed out
    int ioff, joff;          // added to emitted indices
    // Bucketed mode (the LSH join): the rows of P and Q have been regrouped so that each bucket is a
    // contiguous row range, and the work list names (P row range, Q row range) units instead of the grid.
    const int4 *units;             // per unit: first P row, P rows (<= P_ROWS = 256), first Q row, Q rows
    const unsigned int *nunits;    // number of units (written by the kernel that builds the list)
    const int *perm_p, *perm_q;    // regrouped position -> original row
    const uint4 *rec_p, *rec_q;    // per ORIGINAL row: the 16-bit hash keys of all repetitions, rec_words x 16 bytes
    int rec_words;
    int rep;                       // repetitions already joined: a pair whose keys agreed in one of them is not reported again
    // I8/COS: candidates of the fp32 filter are decided exactly from the rows themselves when they leave the CTA
    const void *rows_p, *rows_q;   // the row arrays the tensor maps cover
    int row_bytes;
    double thr_d;                  // t
    // Variant selection on the device.  With sel_mode != 0 the host launches the plain and the ALT instantiation
    // back to back and each decides from the same two device words whether it is the one to run; the other returns
    // at once.  The host therefore needs no round trip between the pre-pass that writes the words and the join.
    //   SEL_I8_RANGE   words = max|P|, max|Q| over all int8 coordinates: ALT (16-bit epilogue) iff d * max * max <= 32767
    //   SEL_L2_RADIUS  words = float bits of max |x|^2, max |y|^2: ALT (candidates decided from the rows) iff the rounding
    //                  error of the norm expansion, sel_coef * (max|x|^2 + max|y|^2), exceeds 1.9 % of r^2
    const unsigned int *sel_words;
    int sel_mode;
    float sel_coef;
    float thr_hi;                  // row-deciding inner-product / cosine forms: scores above this threshold pass without a look at the rows
    float l2_xscale_hi, l2_ycoef_hi, l2_thr_sure;   // the same for the small-radius Euclidean form: the filter's coefficients, raised
    float sel_r2;                  // SEL_L2_RADIUS: r^2 (the kernel's own threshold differs when it runs on transformed operands)
    // When not null: a 64-byte control block that no launch of this call reads or writes.  The kernel zeroes it, so
    // that the caller's next join finds its counter, status and selection words cleared without a memset of its own.
    unsigned long long *zero_next;
    // When not null: two words of pinned host memory that the device can write.  The last CTA to finish (a ticket in
    // done_ticket, a zeroed word of the control block) stores the pair count and the status word there, which saves
    // the device-to-host copy that would otherwise follow the kernel in the stream.
    unsigned long long *host_result;
    unsigned int *done_ticket;
    // BF16/L2, ALT: the tile test is a filter  s >= (l2_xscale |x|^2 - l2_thr_filter) / 2 + l2_ycoef |y|^2, lowered by the
    // error bound so that every pair the difference form accepts is a candidate
    float l2_xscale, l2_ycoef, l2_thr_filter;
    // KIND_SIGN
    uint32_t *key_out;
    long long key_ld;              // 32-bit words per key record
    // KIND_STORE
    uint16_t *store_out;
    long long store_ld;
    float store_scale;
};

constexpr int SEL_NONE = 0, SEL_I8_RANGE = 1, SEL_L2_RADIUS = 2, SEL_IP_SMALL = 3;
// Share of r^2 that the norm expansion's rounding error may reach before the Euclidean join switches to deciding
// candidates from the rows: the tolerance is |distance - r| <= 1e-2 r, i.e. 1.99 % of r^2 on the squared scale.
constexpr float L2_BAND_SHARE = 0.019f;
// Share of the tolerance band 1e-2 |t| that the fp32 accumulation error of an inner product (at most sel_coef |x| |y|)
// may reach before a bf16 inner-product or cosine join switches to deciding candidates from the rows in fp64.
constexpr float IPCOS_BAND_SHARE = 0.5e-2f;
// How far below the threshold that form's tile filter sits, in units of the error bound.
constexpr float IPCOS_FILTER_MARGIN = 1.25f;
__device__ __forceinline__ bool alt_selected(const JoinParams &p) {
    const unsigned int a = __ldg(p.sel_words), b = __ldg(p.sel_words + 1);
    if (p.sel_mode == SEL_I8_RANGE) return (unsigned long long)p.row_bytes * a * b <= 32767ull;
    // SEL_IP_SMALL: the words hold max |x|^2 and max |y|^2, sel_r2 the threshold t
    if (p.sel_mode == SEL_IP_SMALL) return p.sel_coef * (sqrtf(__uint_as_float(a)) * sqrtf(__uint_as_float(b))) > IPCOS_BAND_SHARE * fabsf(p.sel_r2);
    return p.sel_coef * (__uint_as_float(a) + __uint_as_float(b)) > L2_BAND_SHARE * p.sel_r2;
}

struct Ctrl {
    uint64_t full[MAX_STAGES], empty[MAX_STAGES];
    uint64_t pfull[2], pempty[2];      // P_BUFS of each are used
    uint64_t tfull[2], tempty[2];
    uint64_t drain[2];
    uint32_t tmem_base;
    volatile uint32_t abort;
};
static_assert(sizeof(Ctrl) <= CTRL_BYTES, "control block too large");

// One unit of work: P block `pb` against Q tiles [q0, q1).  Q is cut into panels of `qpanel` tiles
// that fit in L2; within a panel CTAs take whole sweeps in waves of gridDim.x P blocks (all CTAs
// then walk the panel together, so a Q tile is fetched from HBM once and served from L2 to everyone
// else, wave after wave); the last, partial wave of a panel lays its `rem` sweeps end to end and cuts them
// into gridDim.x equal runs, so every CTA gets the same number of tiles (a run that crosses from one sweep
// into the next becomes two units).
struct Unit {
    int pb, q0, q1;
    int prow0, prows, qrow0, qrows;   // bucketed mode only
};
template <bool GROUPED, int TN = TILE_N>
__device__ __forceinline__ bool get_unit(const JoinParams &p, int u, Unit &un) {
    const int G = gridDim.x, c = blockIdx.x;
    if constexpr (GROUPED) {
        // units are listed bucket by bucket, so neighbouring CTAs sweep the same Q rows
        const long long idx = (long long)u * G + c;
        if (idx >= (long long)__ldg(p.nunits)) return false;
        const int4 e = __ldg(p.units + idx);
        un.pb = 0;
        un.q0 = 0;
        un.q1 = (e.w + TN - 1) / TN;
        un.prow0 = e.x; un.prows = e.y; un.qrow0 = e.z; un.qrows = e.w;
        return true;
    }
    if (p.wave_gq > 0) {
        // Very long rows: 148 resident P tiles no longer fit in L2 next to a Q panel, and every tile would come
        // from DRAM.  Instead a wave covers GP P tiles x GQ Q tiles, one pair per CTA; the Q index moves fastest
        // from wave to wave, so the GP P tiles stay in L2 while Q streams through once per row of waves.
        const int GQ = p.wave_gq, GP = G / GQ;
        if (c >= GP * GQ) return false;                         // spare CTAs
        const int a = c / GQ, b = c - a * GQ;
        const int WQ = (p.QT + GQ - 1) / GQ, WP = (p.PB + GP - 1) / GP;
        const int wp = u / WQ, wq = u - wp * WQ;
        if (wp >= WP) return false;
        const int pb = wp * GP + a, qt = wq * GQ + b;
        const bool inside = pb < p.PB && qt < p.QT;             // the edges of the grid leave some pairs empty
        un.pb = inside ? pb : 0;
        un.q0 = inside ? qt : 0;
        un.q1 = inside ? qt + 1 : 0;
        return true;
    }
    const int full = p.PB / G, rem = p.PB - full * G;
    const int per_panel = full + (rem > 0 ? 2 : 0);
    const int panel = u / per_panel, v = u - panel * per_panel;
    const int pq0 = panel * p.qpanel;
    if (pq0 >= p.QT) return false;
    const int pq1 = min(pq0 + p.qpanel, p.QT);
    if (v < full) { un.pb = v * G + c; un.q0 = pq0; un.q1 = pq1; return true; }
    // v == full or full + 1, rem > 0: the partial wave.  This CTA's run is [t0, t1) of the rem * len tiles;
    // it lies in sweep t0 / len and, if it crosses the sweep's end, in the next one (rem <= G: never further).
    const int len = pq1 - pq0;
    const long long T = (long long)rem * len;
    const long long t0 = T * c / G, t1 = T * (c + 1) / G;
    const int sweep = (int)(t0 / len);
    const long long cut = min(t1, (long long)(sweep + 1) * len);
    if (v == full) {
        un.pb = full * G + sweep;
        un.q0 = pq0 + (int)(t0 - (long long)sweep * len);
        un.q1 = pq0 + (int)(cut - (long long)sweep * len);
    } else {
        un.pb = full * G + (cut < t1 ? sweep + 1 : sweep);
        un.q0 = pq0;
        un.q1 = pq0 + (int)(t1 - cut);                          // empty unless the run crossed into the next sweep
    }
    return true;
}

// The k-th tile a CTA visits in its unit.  Every CTA starts its sweep at a different offset and wraps
// around, so that at any moment the CTAs read different Q tiles instead of all hitting the same L2
// lines at once (measured: the aligned sweep is ~5 % slower on two-chunk tiles once Q is L2-resident).
template <bool ALIGNED>
__device__ __forceinline__ int tile_at(const Unit &un, int k) {
    if constexpr (ALIGNED) return un.q0 + k;
    const int len = un.q1 - un.q0;
    int idx = k + (int)((long long)blockIdx.x * len / gridDim.x);
    if (idx >= len) idx -= len;
    return un.q0 + idx;
}

// Bounded wait on an mbarrier phase.  Returns false when the CTA is aborting.  The hot loop is a
// bare try_wait (the hardware suspends the thread inside it); the abort flag and the cycle budget
// are only looked at every 256 failed attempts so that they stay off the critical path.
__device__ __forceinline__ bool wait_bar(uint64_t *bar, uint32_t parity, Ctrl *ctrl, unsigned int *status, uint32_t site,
                                         long long limit = WAIT_LIMIT_CYCLES) {
    const uint32_t addr = smem_u32(bar);
    long long t0 = 0;
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(addr, parity)) return true;
        if ((it & 0xFF) == 0) {
            if (ctrl->abort) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            if (now - t0 > limit) {
                ctrl->abort = 1;
                atomicCAS(status, 0u, 0x80000000u | site);
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool wait_bar_warp(uint64_t *bar, uint32_t parity, Ctrl *ctrl, unsigned int *status, uint32_t site) {
    const bool ok = wait_bar(bar, parity, ctrl, status, site);
    return __all_sync(0xffffffffu, ok);
}

// One TMEM load of a warp's EPI_COLS columns: 32-bit words, or two 16-bit columns per word.
__device__ __forceinline__ void tmem_ld_words(uint32_t taddr, uint32_t (&v)[128], std::false_type) { tmem_ld_32x32_x128(taddr, v); }
__device__ __forceinline__ void tmem_ld_words(uint32_t taddr, uint32_t (&v)[64], std::false_type) { tmem_ld_32x32_x64(taddr, v); }
__device__ __forceinline__ void tmem_ld_words(uint32_t taddr, uint32_t (&v)[64], std::true_type) { tmem_ld_32x32_x64_pack16(taddr, v); }
__device__ __forceinline__ void tmem_ld_words(uint32_t taddr, uint32_t (&v)[32], std::true_type) { tmem_ld_32x32_x32_pack16(taddr, v); }

// Tree maximum over N accumulator words (3-input max per step keeps the dependency chain at
// log3(N) instead of N).  MODE 0: fp32, 1: int32, 2: two signed 16-bit values per word.
constexpr int MAX_F32 = 0, MAX_S32 = 1, MAX_S16X2 = 2;
template <int MODE>
__device__ __forceinline__ uint32_t max3_words(uint32_t a, uint32_t b, uint32_t c) {
    if constexpr (MODE == MAX_S32) return (uint32_t)__vimax3_s32((int)a, (int)b, (int)c);
    else if constexpr (MODE == MAX_S16X2) return __vimax3_s16x2(a, b, c);
    else return __float_as_uint(fmaxf(fmaxf(__uint_as_float(a), __uint_as_float(b)), __uint_as_float(c)));
}
template <int N, int MODE>
struct TreeMax {
    static __device__ __forceinline__ uint32_t run(const uint32_t *a) {
        constexpr int M = (N + 2) / 3;
        uint32_t t[M];
#pragma unroll
        for (int c = 0; c < M; ++c) {
            if (3 * c + 2 < N) t[c] = max3_words<MODE>(a[3 * c], a[3 * c + 1], a[3 * c + 2]);
            else if (3 * c + 1 < N) t[c] = max3_words<MODE>(a[3 * c], a[3 * c + 1], a[3 * c + 1]);
            else t[c] = a[3 * c];
        }
        return TreeMax<M, MODE>::run(t);
    }
};
template <int MODE>
struct TreeMax<1, MODE> {
    static __device__ __forceinline__ uint32_t run(const uint32_t *a) { return a[0]; }
};

// Write `fill` staged pairs of this warp to the output list: one atomic reserves the slots, the
// stores are coalesced.
// Bucketed mode, repetition > 0: did the hash keys of regrouped rows (i, j) already agree in an earlier
// repetition?  Then that repetition found and reported the pair (Section 4's union over repetitions).
// The key records stay in the rows' original order and are reached through the regrouping permutation: one more
// dependent load per staged pair, against two gathers of all key records per repetition.
__device__ __forceinline__ bool already_reported(const JoinParams &p, long long i, long long j) {
    const uint4 *rp = p.rec_p + (long long)__ldg(p.perm_p + i) * p.rec_words, *rq = p.rec_q + (long long)__ldg(p.perm_q + j) * p.rec_words;
    bool seen = false;
    for (int w = 0; w * 8 < p.rep; ++w) {
        const uint4 a = __ldg(rp + w), b = __ldg(rq + w);
        const uint32_t x[4] = {a.x ^ b.x, a.y ^ b.y, a.z ^ b.z, a.w ^ b.w};
#pragma unroll
        for (int h = 0; h < 8; ++h) {
            const uint32_t diff = (h & 1) ? (x[h >> 1] >> 16) : (x[h >> 1] & 0xffffu);
            seen = seen || (w * 8 + h < p.rep && diff == 0);
        }
    }
    return seen;
}

// I8/COS: the exact decision for the pair of rows (li of P, lj of Q), from the rows themselves.  <x,y>, |x|^2,
// |y|^2 are exact integers, the product |x|^2 |y|^2 an exact 64-bit integer; then three fp64 roundings -- the
// integer to double, the square root, the quotient -- and the compare with t.  A zero vector scores 0.
__device__ __forceinline__ bool cos_i8_passes(const JoinParams &p, long long li, long long lj) {
    const int g = p.row_bytes >> 4;
    const uint4 *x = reinterpret_cast<const uint4 *>(static_cast<const char *>(p.rows_p) + li * p.row_bytes);
    const uint4 *y = reinterpret_cast<const uint4 *>(static_cast<const char *>(p.rows_q) + lj * p.row_bytes);
    int s = 0, nx = 0, ny = 0;
    for (int c = 0; c < g; ++c) {
        const uint4 a = __ldg(x + c), b = __ldg(y + c);
        s = __dp4a((int)a.x, (int)b.x, s);   nx = __dp4a((int)a.x, (int)a.x, nx);   ny = __dp4a((int)b.x, (int)b.x, ny);
        s = __dp4a((int)a.y, (int)b.y, s);   nx = __dp4a((int)a.y, (int)a.y, nx);   ny = __dp4a((int)b.y, (int)b.y, ny);
        s = __dp4a((int)a.z, (int)b.z, s);   nx = __dp4a((int)a.z, (int)a.z, nx);   ny = __dp4a((int)b.z, (int)b.z, ny);
        s = __dp4a((int)a.w, (int)b.w, s);   nx = __dp4a((int)a.w, (int)a.w, nx);   ny = __dp4a((int)b.w, (int)b.w, ny);
    }
    if (nx == 0 || ny == 0) return 0.0 >= p.thr_d;
    const double den = __dsqrt_rn(__ll2double_rn((long long)nx * (long long)ny));
    return __ddiv_rn((double)s, den) >= p.thr_d;
}

// BF16/L2, small radii: the decision for the pair of rows (li of P, lj of Q) in the difference form
// sum (x_k - y_k)^2 <= r^2, fp32, which does not cancel the way |x|^2 + |y|^2 - 2<x,y> does when r^2 is far
// below the norms (relative error about d * 2^-24 whatever the radius).
__device__ __forceinline__ bool l2_bf16_passes(const JoinParams &p, long long li, long long lj) {
    const int g = p.row_bytes >> 4;
    const uint4 *x = reinterpret_cast<const uint4 *>(static_cast<const char *>(p.rows_p) + li * p.row_bytes);
    const uint4 *y = reinterpret_cast<const uint4 *>(static_cast<const char *>(p.rows_q) + lj * p.row_bytes);
    float s[4] = {0.f, 0.f, 0.f, 0.f};
    for (int c = 0; c < g; ++c) {
        const uint4 a = __ldg(x + c), b = __ldg(y + c);
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const float e0 = __uint_as_float(aw[t] << 16) - __uint_as_float(bw[t] << 16);
            const float e1 = __uint_as_float(aw[t] & 0xffff0000u) - __uint_as_float(bw[t] & 0xffff0000u);
            s[t] = fmaf(e0, e0, s[t]);
            s[t] = fmaf(e1, e1, s[t]);
        }
    }
    return (s[0] + s[1]) + (s[2] + s[3]) <= p.thr_f;
}

// BF16 inner product / cosine, thresholds so close to zero that the tolerance band is narrower than the fp32 accumulation
// error: the decision for the pair of rows (li of P, lj of Q) in fp64 -- products of bf16 values are exact in fp64, the
// sums run over k ascending, the cosine is <x,y> / (sqrt(|x|^2) sqrt(|y|^2)) and 0 for a zero vector; the compare takes
// the fp64 threshold.
template <bool COS>
__device__ __forceinline__ bool ipcos_bf16_passes(const JoinParams &p, long long li, long long lj) {
    const int g = p.row_bytes >> 4;
    const uint4 *x = reinterpret_cast<const uint4 *>(static_cast<const char *>(p.rows_p) + li * p.row_bytes);
    const uint4 *y = reinterpret_cast<const uint4 *>(static_cast<const char *>(p.rows_q) + lj * p.row_bytes);
    double s = 0.0, nx = 0.0, ny = 0.0;
    for (int c = 0; c < g; ++c) {
        const uint4 a = __ldg(x + c), b = __ldg(y + c);
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const double x0 = (double)__uint_as_float(aw[t] << 16), x1 = (double)__uint_as_float(aw[t] & 0xffff0000u);
            const double y0 = (double)__uint_as_float(bw[t] << 16), y1 = (double)__uint_as_float(bw[t] & 0xffff0000u);
            s = __dadd_rn(s, __dmul_rn(x0, y0));
            s = __dadd_rn(s, __dmul_rn(x1, y1));
            if constexpr (COS) {
                nx = __dadd_rn(nx, __dmul_rn(x0, x0));
                nx = __dadd_rn(nx, __dmul_rn(x1, x1));
                ny = __dadd_rn(ny, __dmul_rn(y0, y0));
                ny = __dadd_rn(ny, __dmul_rn(y1, y1));
            }
        }
    }
    if constexpr (COS) {
        if (nx == 0.0 || ny == 0.0) return 0.0 >= p.thr_d;
        return __ddiv_rn(s, __dmul_rn(__dsqrt_rn(nx), __dsqrt_rn(ny))) >= p.thr_d;
    }
    return s >= p.thr_d;
}

// Is the staged pair dropped when it leaves the CTA?  Bucketed mode: reported by an earlier repetition.  VERIFY:
// the pair is a candidate of a tile-level filter and fails the decision taken from its two rows (VERIFY_COS_I8: the
// exact int8 cosine; VERIFY_L2_BF16: the difference-form Euclidean test).  Staged indices are regrouped positions
// in bucketed mode, else row indices plus the caller's offsets.
constexpr int VERIFY_NONE = 0, VERIFY_COS_I8 = 1, VERIFY_L2_BF16 = 2, VERIFY_IP_BF16 = 3, VERIFY_COS_BF16 = 4;
// The bf16 kinds (VERIFY_L2_BF16, VERIFY_IP_BF16, VERIFY_COS_BF16) stage a candidate with bit 31 of j set and a pair that is sure to pass with the bit
// clear: only candidates are decided from their rows (`candidate`; the other kinds decide every staged pair).
__host__ __device__ constexpr bool verify_flags(int verify) { return verify == 2 || verify == 3 || verify == 4; }
template <bool GROUPED, int VERIFY>
__device__ __forceinline__ bool drop_pair(const JoinParams &p, int i, int j, bool candidate = true) {
    if constexpr (GROUPED) {
        if (p.rep > 0 && already_reported(p, i, j)) return true;
    }
    if (verify_flags(VERIFY) && !candidate) return false;
    if constexpr (VERIFY == VERIFY_COS_I8) {
        if (!cos_i8_passes(p, GROUPED ? i : i - p.ioff, GROUPED ? j : j - p.joff)) return true;
    }
    if constexpr (VERIFY == VERIFY_L2_BF16) {
        if (!l2_bf16_passes(p, GROUPED ? i : i - p.ioff, GROUPED ? j : j - p.joff)) return true;
    }
    if constexpr (VERIFY == VERIFY_IP_BF16 || VERIFY == VERIFY_COS_BF16) {
        if (!ipcos_bf16_passes<VERIFY == VERIFY_COS_BF16>(p, GROUPED ? i : i - p.ioff, GROUPED ? j : j - p.joff)) return true;
    }
    return false;
}

template <bool GROUPED>
__device__ __forceinline__ int2 final_pair(const JoinParams &p, int2 pr) {
    if constexpr (GROUPED) return make_int2(__ldg(p.perm_p + pr.x) + p.ioff, __ldg(p.perm_q + pr.y) + p.joff);
    return pr;
}
// Write `count` staged pairs to out[base ..]: all 32 lanes together, consecutive slots.  Bucketed mode turns regrouped
// positions into rows on the way (two dependent lookups per pair): the lookups of up to six pairs per lane (a whole staging buffer per pass) are issued
// before the first store, so that their latencies overlap instead of adding up (a dense bucketed join spends most of
// its time here).
template <bool GROUPED>
__device__ __forceinline__ void write_staged(const JoinParams &p, const int2 *buf, int count, unsigned long long base, int lane) {
    constexpr int U = 6;
    for (int k0 = 0; k0 < count; k0 += 32 * U) {
        int2 fp[U];
#pragma unroll
        for (int t = 0; t < U; ++t) {
            const int k = k0 + 32 * t + lane;
            fp[t] = k < count ? final_pair<GROUPED>(p, buf[k]) : make_int2(0, 0);
        }
#pragma unroll
        for (int t = 0; t < U; ++t) {
            const int k = k0 + 32 * t + lane;
            const unsigned long long slot = base + (unsigned long long)k;
            if (k < count && slot < p.capacity) p.out[slot] = fp[t];
        }
    }
}

template <bool GROUPED, int VERIFY = VERIFY_NONE>
__device__ __forceinline__ void flush_pairs(const JoinParams &p, const int2 *buf, int fill, int lane) {
    if (fill == 0) return;
    if constexpr (GROUPED || VERIFY != VERIFY_NONE) {
        if (VERIFY != VERIFY_NONE || p.rep > 0) {
            // Duplicates (and, for the filtered kinds, candidates that fail the exact test) are dropped here, a whole buffer
            // at a time (32 lookups in flight per step), not when a hit is found: there the lookup's latency
            // would stall the CTA's pipeline.
            int2 *wbuf = const_cast<int2 *>(buf);
            int kept = 0;
            for (int k0 = 0; k0 < fill; k0 += 32) {
                const int k = k0 + lane;
                bool keep = false;
                if (k < fill) {
                    int2 pr = wbuf[k];
                    bool candidate = true;
                    if constexpr (verify_flags(VERIFY)) {
                        candidate = pr.y < 0;
                        pr.y &= 0x7fffffff;
                        wbuf[k].y = pr.y;
                    }
                    keep = !drop_pair<GROUPED, VERIFY>(p, pr.x, pr.y, candidate);
                    if (!keep) wbuf[k].x = -1;
                }
                kept += __popc(__ballot_sync(0xffffffffu, keep));
            }
            unsigned long long base = 0;
            if (lane == 0 && kept) base = atomicAdd(p.counter, (unsigned long long)kept);
            base = __shfl_sync(0xffffffffu, base, 0);
            __syncwarp();
            int run = 0;
            for (int k0 = 0; k0 < fill; k0 += 32) {
                const int k = k0 + lane;
                const int2 pr = k < fill ? wbuf[k] : make_int2(-1, 0);
                const bool keep = pr.x >= 0;
                const uint32_t b = __ballot_sync(0xffffffffu, keep);
                const unsigned long long slot = base + (unsigned long long)(run + __popc(b & ((1u << lane) - 1u)));
                if (keep && slot < p.capacity) p.out[slot] = final_pair<GROUPED>(p, pr);
                run += __popc(b);
            }
            __syncwarp();
            return;
        }
    }
    unsigned long long base = 0;
    if (lane == 0) base = atomicAdd(p.counter, (unsigned long long)fill);
    base = __shfl_sync(0xffffffffu, base, 0);
    __syncwarp();
    write_staged<GROUPED>(p, buf, fill, base, lane);
    __syncwarp();
}

// Compact the pairs (i, j0 + 32*q + c), c in mask[q], of the 32 rows this warp owns: popcount
// prefix over the warp, then into the warp's shared-memory staging buffer, which is flushed with
// one global atomic per ~STAGE_PAIRS pairs.  A block with more hits than the buffer holds leaves in
// rounds through the same buffer.  `fill` (warp-uniform) is the number of pairs staged so far.
// `cand` (kinds with verify_flags only): the columns of `mask` that are candidates; their staged j carries bit 31.
template <int NQ, bool GROUPED, int VERIFY = VERIFY_NONE, int SP = STAGE_PAIRS>
__device__ __forceinline__ void emit_pairs(const JoinParams &p, const uint32_t (&mask)[NQ], int lane, long long i, long long j0,
                                           int2 *buf, int &fill, const uint32_t *cand = nullptr) {
    constexpr bool FLAGS = verify_flags(VERIFY);
    auto flag_of = [&](int q, int c) -> int { return FLAGS ? (int)(((cand[q] >> c) & 1u) << 31) : 0; };
    int cnt = 0;
#pragma unroll
    for (int q = 0; q < NQ; ++q) cnt += __popc(mask[q]);
    // prefix sum over the lanes.  Usual case, at most one hit per row: two votes instead of a chain of shuffles
    int incl, total;
    const uint32_t one = __ballot_sync(0xffffffffu, cnt != 0);
    if (one == 0) return;
    const bool single = __ballot_sync(0xffffffffu, cnt > 1) == 0;
    if (single) {
        incl = __popc(one & (0xffffffffu >> (31 - lane)));
        total = __popc(one);
    } else {
        incl = cnt;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += t;
        }
        total = __shfl_sync(0xffffffffu, incl, 31);
    }
    if (fill + total > SP) {
        flush_pairs<GROUPED, VERIFY>(p, buf, fill, lane);
        fill = 0;
    }
    // bucketed mode stages regrouped positions; they become original rows when they leave the CTA
    const int ii = (int)(i + (GROUPED ? 0 : p.ioff));
    const int jj = (int)(j0 + (GROUPED ? 0 : p.joff));
    if (total > SP) {
        // More hits in one block than the buffer holds (very dense outputs: a low threshold, or the buckets of an LSH
        // join on clustered data, where a quarter of all scores can pass).  The block leaves in rounds through the
        // (empty) staging buffer: every lane contributes up to SP / 32 of its remaining hits per round, and the round is
        // written out by all 32 lanes together -- coalesced stores, the position -> row lookups of bucketed mode 32 in
        // flight -- instead of every lane walking its own hits with one dependent lookup and one 8-byte store each, and
        // one atomic per pair where pairs can be dropped.  Where nothing can be dropped the whole block's slots are
        // reserved with one atomic up front; otherwise every round goes through flush_pairs.
        constexpr int PER_LANE = SP / 32;
        bool plain = true;
        if constexpr (GROUPED || VERIFY != VERIFY_NONE) plain = !(VERIFY != VERIFY_NONE || p.rep > 0);
        unsigned long long base = 0;
        if (plain) {
            if (lane == 0) base = atomicAdd(p.counter, (unsigned long long)total);
            base = __shfl_sync(0xffffffffu, base, 0);
        }
        uint32_t m[NQ];
#pragma unroll
        for (int q = 0; q < NQ; ++q) m[q] = mask[q];
        int remaining = cnt;
        while (__any_sync(0xffffffffu, remaining > 0)) {
            const int take = min(remaining, PER_LANE);
            int inc = take;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, inc, off);
                if (lane >= off) inc += t;
            }
            const int round_total = __shfl_sync(0xffffffffu, inc, 31);
            int pos = inc - take;
            for (int t = 0; t < take; ++t) {
                int col = 0;
                bool found = false;
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    if (!found && m[q] != 0) {
                        const int c = __ffs(m[q]) - 1;
                        col = (32 * q + c) | flag_of(q, c);
                        m[q] &= m[q] - 1;
                        found = true;
                    }
                }
                buf[pos++] = make_int2(ii, (jj + (col & 0x7fffffff)) | (col & (int)0x80000000));
            }
            remaining -= take;
            __syncwarp();
            if (plain) {
                write_staged<GROUPED>(p, buf, round_total, base, lane);
                base += (unsigned long long)round_total;
                __syncwarp();
            } else {
                flush_pairs<GROUPED, VERIFY>(p, buf, round_total, lane);
            }
        }
        return;
    }
    if (single) {
        // one hit per row at most (total <= 32 fits): every hit lane finds its one column without a loop
        if (cnt != 0) {
            int col = 0;
#pragma unroll
            for (int q = 0; q < NQ; ++q)
                if (mask[q] != 0) {
                    const int c = __ffs(mask[q]) - 1;
                    col = (32 * q + c) | flag_of(q, c);
                }
            buf[fill + incl - 1] = make_int2(ii, (jj + (col & 0x7fffffff)) | (col & (int)0x80000000));
        }
        fill += total;
        __syncwarp();
        return;
    }
    int pos = fill + incl - cnt;
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        uint32_t mk = mask[q];
        while (mk) {
            const int c = __ffs(mk) - 1;
            mk &= mk - 1;
            buf[pos++] = make_int2(ii, (jj + 32 * q + c) | flag_of(q, c));
        }
    }
    fill += total;
    __syncwarp();
}

// Store epilogue (KIND_STORE) of one warp: NC accumulator columns (rows of Q = output rows j_first ..) of its 32
// TMEM lanes (rows of P = output coordinates i_base ..) are scaled, rounded to bf16 and transposed through the
// warp's 2 KiB of shared memory, 32 columns at a time, so that every global store is 16 bytes and 4 lanes cover
// the 64 contiguous bytes the warp owns of one output row.
template <int NC>
__device__ __forceinline__ void store_tile_part(const JoinParams &p, uint32_t taddr, uint64_t *tempty_bar, int lane, uint16_t *sb,
                                                long long j_first, long long q_end, int i_base) {
    uint32_t v[NC];
    tmem_ld_words(taddr, v, std::false_type{});
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(tempty_bar));
#pragma unroll
    for (int rnd = 0; rnd < NC / 32; ++rnd) {
#pragma unroll
        for (int c = 0; c < 32; ++c)
            sb[c * 32 + lane] = __bfloat16_as_ushort(__float2bfloat16_rn(__uint_as_float(v[rnd * 32 + c]) * p.store_scale));
        __syncwarp();
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const int q = t * 32 + lane, jl = q >> 2, part = q & 3;
            const uint4 val = *reinterpret_cast<const uint4 *>(sb + jl * 32 + part * 8);
            const long long j = j_first + rnd * 32 + jl;
            const int icol = i_base + part * 8;                        // 8 coordinates: all valid or none (k_i % 8 == 0)
            if (j < q_end && icol < (int)p.n) *reinterpret_cast<uint4 *>(p.store_out + j * p.store_ld + icol) = val;
        }
        __syncwarp();
    }
}

// The MMA-issuing role (warps 1 and 3).  KC > 0 is a fast path with the chunks per tile known at
// compile time (resident P block, full 128-byte chunks, two issuers): measured on B200, a chunk loop
// with a run-time trip count around the tcgen05.mma issues costs ~80 cycles per tile, the run-time
// operand-address select another ~25.  KC == 0 is the general path.
// ONE_BLOCK_OK: a tile whose second P block lies wholly past the end of P skips that block's MMAs (the store
// kind, whose resident operand often has <= 128 rows; the join kinds keep the branch out of their issue loop).
// WIDEQ: one resident block against 256 streamed rows (N = 256); the second block is never issued.
// LASTK (fast path only): 32-byte K steps issued for a tile's last chunk -- 4 for rows of whole chunks; fewer where the
// rest of the chunk is known to be zero (the transformed operands of dense Euclidean joins end 16 bytes into their
// last chunk), which saves the tensor work and the energy of multiplying zeros.
// SPLIT (fast path only): both issuing warps work on every tile, warp 1 on P block 0 and warp 3 on P block 1, and wait
// for the tile's operand chunks before they wait for the accumulator.  The time from an accumulator's hand-back to its
// next commit then holds one barrier wait and half a tile's issues instead of three waits and a whole tile's -- for the
// epilogue whose warp groups own one accumulator each, where that time is not hidden behind another tile's tests.
template <int DT, int KC, bool GROUPED, bool ONE_BLOCK_OK, bool WIDEQ = false, int LASTK = 4, bool SPLIT = false>
__device__ __forceinline__ void mma_issuer_role(const JoinParams &p, Ctrl *ctrl, uint8_t *smem_p, uint8_t *smem_ring,
                                                const int stage_bytes_rt, const uint32_t tmem_base, const int warp, const int lane) {
    constexpr bool FAST = KC > 0;
    static_assert(!SPLIT || (FAST && !WIDEQ), "split issue: compile-time chunk count, standard geometry");
    constexpr uint32_t idesc = umma_idesc(DT == DT_I8 ? 2u : 1u, 1u, TILE_M, WIDEQ ? LONG_TN : TILE_N);
    const int kc = FAST ? KC : p.kc;
    const bool stationary = FAST ? true : p.stationary != 0;
    const bool epi_release = FAST ? true : p.epi_release != 0;
    const int stage_bytes = FAST ? B_CHUNK_BYTES : stage_bytes_rt;
    const bool dual = epi_release;
    const uint32_t mid = warp == 1 ? 0u : 1u;
    uint32_t stage = 0, phase = 0, pbuf = 0, pphase = 0, tsel = 0;
    uint32_t accph0 = 0, accph1 = 0;            // phase of each accumulator's hand-back barrier
    bool ok = true;
    Unit un;
    for (int u = 0; ok && (dual || mid == 0) && get_unit<GROUPED>(p, u, un); ++u) {
        if (un.q1 <= un.q0) continue;
        if (stationary) {
            ok = wait_bar_warp(&ctrl->pfull[pbuf], pphase, ctrl, p.status, 3);
            if (!ok) break;
        }
        const bool two = !WIDEQ && (!ONE_BLOCK_OK || (GROUPED ? un.prows > TILE_M : (long long)un.pb * P_ROWS + TILE_M < p.n));
        for (int k = 0; ok && k < un.q1 - un.q0; ++k, tsel ^= 1) {
            if (!SPLIT && dual && tsel != mid) {
                // the other issuer's tile: step over its chunks in the ring
                stage += (uint32_t)kc;
                while (stage >= (uint32_t)p.nstages) { stage -= (uint32_t)p.nstages; phase ^= 1; }
                continue;
            }
            const uint32_t a = tsel;                       // accumulator of this tile
            const uint32_t d_tmem = tmem_base + a * ACC_COLS;
            if constexpr (SPLIT) {
                uint32_t st = stage, ph = phase;
#pragma unroll
                for (int c = 0; c < KC; ++c) {
                    ok = ok && wait_bar_warp(&ctrl->full[st], ph, ctrl, p.status, 5);
                    if (++st == (uint32_t)p.nstages) { st = 0; ph ^= 1; }
                }
                if (!ok) break;
            }
            ok = wait_bar_warp(&ctrl->tempty[a], (a ? accph1 : accph0) ^ 1, ctrl, p.status, 4);
            if (!ok) break;
#pragma unroll
            for (int c = 0; c < (FAST ? KC : kc); ++c) {
                if constexpr (!SPLIT) {
                    ok = wait_bar_warp(&ctrl->full[stage], phase, ctrl, p.status, 5);
                    if (!ok) break;
                }
                tc_fence_after();
                // operands are computed by the whole (converged) warp so that they stay warp-uniform;
                // the four K steps are unrolled: a loop around single tcgen05.mma issues is slow
                uint8_t *sb = smem_ring + (size_t)stage * stage_bytes;
                const uint32_t a_addr = stationary ? smem_u32(smem_p + (size_t)(pbuf * kc + c) * A_CHUNK_BYTES)
                                                   : smem_u32(sb + B_CHUNK_BYTES);
                const uint64_t adesc = umma_desc_sw128_kmajor(a_addr);                       // P block 0
                const uint64_t adesc1 = umma_desc_sw128_kmajor(a_addr + A_SUB_BYTES);        // P block 1
                const uint64_t bdesc = umma_desc_sw128_kmajor(smem_u32(sb));
                const bool last_chunk = c == kc - 1;
                const int ksteps = FAST ? ((KC > 0 && c == KC - 1) ? LASTK : 4) : (last_chunk ? p.last_ksteps : 4);
                if (elect_one()) {
                    // the Q chunk against both resident P blocks: block s accumulates in columns s * TILE_N ..
                    if (!SPLIT || mid == 0) {
                        umma_ss<DT == DT_I8>(d_tmem, adesc, bdesc, idesc, c != 0 ? 1u : 0u);
                        if (ksteps > 1) umma_ss<DT == DT_I8>(d_tmem, adesc + 2, bdesc + 2, idesc, 1u);
                        if (ksteps > 2) umma_ss<DT == DT_I8>(d_tmem, adesc + 4, bdesc + 4, idesc, 1u);
                        if (ksteps > 3) umma_ss<DT == DT_I8>(d_tmem, adesc + 6, bdesc + 6, idesc, 1u);
                    }
                    if (two && (!SPLIT || mid == 1)) {
                        umma_ss<DT == DT_I8>(d_tmem + TILE_N, adesc1, bdesc, idesc, c != 0 ? 1u : 0u);
                        if (ksteps > 1) umma_ss<DT == DT_I8>(d_tmem + TILE_N, adesc1 + 2, bdesc + 2, idesc, 1u);
                        if (ksteps > 2) umma_ss<DT == DT_I8>(d_tmem + TILE_N, adesc1 + 4, bdesc + 4, idesc, 1u);
                        if (ksteps > 3) umma_ss<DT == DT_I8>(d_tmem + TILE_N, adesc1 + 6, bdesc + 6, idesc, 1u);
                    }
                    if (!epi_release) umma_commit(smem_u32(&ctrl->empty[stage]));
                    if (last_chunk) umma_commit(smem_u32(&ctrl->tfull[a]));
                }
                __syncwarp();
                if (++stage == (uint32_t)p.nstages) { stage = 0; phase ^= 1; }
            }
            if (!ok) break;
            if (a) accph1 ^= 1; else accph0 ^= 1;
        }
        if (ok && stationary) {
            // the P block may be overwritten once the MMAs of every issuer have retired
            if (elect_one()) umma_commit(smem_u32(&ctrl->pempty[pbuf]));
            __syncwarp();
            if (++pbuf == (uint32_t)p_bufs(GROUPED, kc)) { pbuf = 0; pphase ^= 1; }
        }
    }
    if (!ok) {
        // aborting: wait (bounded) until the MMAs already issued have retired
        if (lane == 0) {
            umma_commit(smem_u32(&ctrl->drain[mid]));
            const long long t0 = clock64();
            while (!mbar_try_wait(smem_u32(&ctrl->drain[mid]), 0) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
        }
        __syncwarp();
    }
}

// Long rows (LONGK): 256 x 256 tiles with one accumulator buffer.  Nothing is resident: every ring stage
// carries a 32 KiB chunk of the Q tile and a 32 KiB chunk of the P tile, and one warp issues 2 x 4 tcgen05.mma
// of N = 256 per chunk (1024 tensor cycles), block s accumulating in TMEM columns s * 256 ...  Per unit of work
// that is 64 KiB of operand traffic per 1024 tensor cycles instead of the 48 KiB per 552 of the streamed
// 256 x 128 tile, and the accumulator hand-off is paid once per K loop.
template <int DT, bool GROUPED>
__device__ __forceinline__ void mma_issuer_long(const JoinParams &p, Ctrl *ctrl, uint8_t *smem_ring, const uint32_t tmem_base,
                                                const int lane) {
    constexpr uint32_t idesc = umma_idesc(DT == DT_I8 ? 2u : 1u, 1u, TILE_M, LONG_TN);
    uint32_t stage = 0, phase = 0, accph = 0;
    bool ok = true;
    Unit un;
    for (int u = 0; ok && get_unit<GROUPED, LONG_TN>(p, u, un); ++u) {
        if (un.q1 <= un.q0) continue;
        for (int k = 0; ok && k < un.q1 - un.q0; ++k) {
            ok = wait_bar_warp(&ctrl->tempty[0], accph ^ 1, ctrl, p.status, 4);
            if (!ok) break;
            for (int c = 0; c < p.kc; ++c) {
                ok = wait_bar_warp(&ctrl->full[stage], phase, ctrl, p.status, 5);
                if (!ok) break;
                tc_fence_after();
                uint8_t *sb = smem_ring + (size_t)stage * LONG_STAGE_BYTES;
                const uint64_t bdesc = umma_desc_sw128_kmajor(smem_u32(sb));
                const uint64_t adesc = umma_desc_sw128_kmajor(smem_u32(sb + LONG_Q_CHUNK_BYTES));
                const uint64_t adesc1 = umma_desc_sw128_kmajor(smem_u32(sb + LONG_Q_CHUNK_BYTES + A_SUB_BYTES));
                const bool last_chunk = c == p.kc - 1;
                const int ksteps = last_chunk ? p.last_ksteps : 4;
                if (elect_one()) {
                    umma_ss<DT == DT_I8>(tmem_base, adesc, bdesc, idesc, c != 0 ? 1u : 0u);
                    if (ksteps > 1) umma_ss<DT == DT_I8>(tmem_base, adesc + 2, bdesc + 2, idesc, 1u);
                    if (ksteps > 2) umma_ss<DT == DT_I8>(tmem_base, adesc + 4, bdesc + 4, idesc, 1u);
                    if (ksteps > 3) umma_ss<DT == DT_I8>(tmem_base, adesc + 6, bdesc + 6, idesc, 1u);
                    umma_ss<DT == DT_I8>(tmem_base + LONG_TN, adesc1, bdesc, idesc, c != 0 ? 1u : 0u);
                    if (ksteps > 1) umma_ss<DT == DT_I8>(tmem_base + LONG_TN, adesc1 + 2, bdesc + 2, idesc, 1u);
                    if (ksteps > 2) umma_ss<DT == DT_I8>(tmem_base + LONG_TN, adesc1 + 4, bdesc + 4, idesc, 1u);
                    if (ksteps > 3) umma_ss<DT == DT_I8>(tmem_base + LONG_TN, adesc1 + 6, bdesc + 6, idesc, 1u);
                    umma_commit(smem_u32(&ctrl->empty[stage]));
                    if (last_chunk) umma_commit(smem_u32(&ctrl->tfull[0]));
                }
                __syncwarp();
                if (++stage == (uint32_t)LONG_STAGES) { stage = 0; phase ^= 1; }
            }
            accph ^= 1;
        }
    }
    if (!ok) {
        if (lane == 0) {
            umma_commit(smem_u32(&ctrl->drain[0]));
            const long long t0 = clock64();
            while (!mbar_try_wait(smem_u32(&ctrl->drain[0]), 0) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
        }
        __syncwarp();
    }
}

// ALT selects the second instantiation of a (element type, kind) pair; which of the two runs is decided on the
// device (JoinParams::sel_mode), or by the host where no selection is in force.
//   int8 (NARROW): every score provably fits in 16 bits, so the epilogue loads the accumulator packed two columns per
//     register and reduces it with packed 16-bit max -- half the registers and half the ALU work of the 32-bit path,
//     which is what bounds short-K tiles.
//   bf16 Euclidean: the radius is too small for the norm expansion |x|^2 + |y|^2 - 2<x,y> in fp32 (its rounding error
//     exceeds the stated tolerance on r): the tile test becomes a filter, lowered by the error bound, and every
//     candidate is decided in the difference form from its two rows when it leaves the CTA.
// KC > 0 (1 or 2): the chunks per tile, and with them the resident-P mode, the ring depth and the
// epilogue hand-back, are compile-time constants -- the host selects these instantiations when the
// run-time values agree.  Measured on B200: -6 % on the one-chunk int8 join.  KC == 0: all run-time.
__host__ __device__ constexpr int fast_nstages(int kc, int pbufs) {
    return (232448 - 1024 - CTRL_BYTES - STAGING_BYTES - pbufs * kc * A_CHUNK_BYTES) / B_CHUNK_BYTES > MAX_STAGES
               ? MAX_STAGES
               : (232448 - 1024 - CTRL_BYTES - STAGING_BYTES - pbufs * kc * A_CHUNK_BYTES) / B_CHUNK_BYTES;
}
// GROUPED: bucketed mode (every element type and kind) -- see JoinParams::units.
// GEO selects the tile geometry.  GEO_LONG: the long-row geometry above (join kinds, brute-force schedule only).
// GEO_WIDEQ (store kind, resident operand of at most 128 rows): one resident block against 256 streamed rows per
// tile -- 4 MMAs of N = 256 per chunk into the 256 columns of an accumulator buffer, 32 KiB TMA transactions --
// which this HBM-bound use prefers to two half-empty 128-column blocks.  In both, mapQ has 256-row boxes.
constexpr int GEO_STD = 0, GEO_LONG = 1, GEO_WIDEQ = 2;
template <int DT, int KIND, bool ALT = false, int KC = 0, bool GROUPED = false, int GEO = GEO_STD, int EW = NUM_EPI_WARPS, int LASTK = 4>
__global__ void __launch_bounds__(num_threads(EW), 1)
join_kernel(const __grid_constant__ CUtensorMap mapP, const __grid_constant__ CUtensorMap mapQ, const JoinParams p_in) {
    constexpr bool LONGK = GEO == GEO_LONG, WIDEQ = GEO == GEO_WIDEQ;
    constexpr bool NARROW = DT == DT_I8 && ALT;
    constexpr bool L2_FILTER = DT == DT_BF16 && KIND == KIND_L2 && ALT;
    // bf16 inner product, ALT: the threshold is zero and folded into the operands (dense joins of every kind on transformed
    // operands), so a score passes when its sign bit is clear -- the element test is one funnel shift, no add.  In the
    // device-side choice between the two Euclidean forms this kernel stands for the plain one.
    constexpr bool IP_SIGN = DT == DT_BF16 && KIND == KIND_IP && ALT && EW == 2 * NUM_EPI_WARPS;
    // bf16 inner product (8 epilogue warps) and cosine, ALT: the tile test is a filter lowered by the fp32 accumulation error
    // bound, and every candidate is decided from its rows in fp64 when the warp's staging buffer is flushed -- for
    // thresholds whose tolerance band 1e-2 |t| is narrower than that error (t = 0 above all).
    constexpr bool IPCOS_FILTER = DT == DT_BF16 && ALT && ((KIND == KIND_IP && EW == NUM_EPI_WARPS) || KIND == KIND_COS);
    constexpr bool SEL_ALT = ALT && !IP_SIGN;
    // The sign test with 16 epilogue warps: the two groups of eight take alternate tiles (group g owns accumulator g), and
    // every warp tests all 128 columns of its 32 rows in two loads of 64, so the per-tile work of a warp (barrier wait,
    // hand-back, tail mask, compaction) is paid once per 128 columns instead of once per 64.
    constexpr bool TWO_TILE = IP_SIGN && EW == 2 * NUM_EPI_WARPS;
    static_assert(DT == DT_I8 || !ALT || KIND == KIND_L2 || KIND == KIND_IP || KIND == KIND_COS, "bf16: the join kinds have a second variant");
    // not the variant the data calls for: the other launch does the work (uniform over the grid, before any barrier
    // or tensor-memory allocation exists)
    if (p_in.zero_next != nullptr && blockIdx.x == 0 && threadIdx.x < 8) p_in.zero_next[threadIdx.x] = 0ull;
    if (p_in.sel_mode != SEL_NONE && alt_selected(p_in) != SEL_ALT) return;
    static_assert(!LONGK || (KC == 0 && KIND != KIND_STORE && KIND != KIND_SIGN), "long-row mode: general join kinds only");
    static_assert(KIND != KIND_SIGN || (KC == 0 && !GROUPED && GEO == GEO_STD && !ALT), "hash keys: general path only");
    static_assert(!WIDEQ || (KC == 0 && !GROUPED && KIND == KIND_STORE), "wide-Q mode: store kind only");
    static_assert(LASTK == 4 || (KC > 0 && LASTK >= 1 && LASTK < 4), "a short last chunk: compile-time chunk counts only");
    static_assert(EW == NUM_EPI_WARPS || (EW == 2 * NUM_EPI_WARPS && GEO == GEO_STD && KIND != KIND_STORE && KIND != KIND_SIGN), "16 epilogue warps: join kinds, standard geometry");
    constexpr int TN = (LONGK || WIDEQ) ? LONG_TN : TILE_N;   // rows of Q per tile
    constexpr int NPASS = TN / TILE_N;                     // 128-column passes of the epilogue over a P block's columns
    constexpr int ECOLS = epi_cols(EW);                    // accumulator columns per epilogue warp and pass
    constexpr int SPAIRS = stage_pairs(EW);                // pairs a warp stages before it flushes
    JoinParams p = p_in;
    if constexpr (IPCOS_FILTER && KIND == KIND_IP) {
        // the filter threshold: t lowered by the error bound at the largest norms (the words hold max |x|^2, max |y|^2)
        const float mx = sqrtf(__uint_as_float(__ldg(p.sel_words))), my = sqrtf(__uint_as_float(__ldg(p.sel_words + 1)));
        const float margin = __fmul_ru(IPCOS_FILTER_MARGIN * p.sel_coef, __fmul_ru(mx, my));
        p.thr_hi = __fadd_ru(p.thr_f, margin);      // above it a score passes whatever its rounding error
        p.thr_f = __fsub_rd(p.thr_f, margin);
    }
    if constexpr (LONGK) {
        p.stationary = 0;
        p.epi_release = 0;
        p.nstages = LONG_STAGES;
    }
    if constexpr (KC > 0) {
        p.kc = KC;
        p.stationary = 1;
        p.epi_release = 1;
        p.nstages = fast_nstages(KC, p_bufs(GROUPED, KC));
        p.last_ksteps = 4;        // (the issuers of a LASTK < 4 instantiation stop short of the chunk's zero-filled rest)
    }
    // Aligned sweeps (no per-CTA rotation): bucketed units are short, and the store kind reads the streamed
    // operand once per 256-row tile of the resident one -- the CTAs that share a segment then walk it in
    // step, so that the second reader finds the tile in L2 (measured: rotated, that level read its input twice).
    constexpr bool ALIGNED = GROUPED || KIND == KIND_STORE || KIND == KIND_SIGN;
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment: the 128-byte swizzle pattern repeats every 1024 bytes.
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kc = p.kc;
    const int p_bytes = p.stationary ? p_bufs(GROUPED, kc) * kc * A_CHUNK_BYTES : 0;
    const int stage_bytes = LONGK ? LONG_STAGE_BYTES : (WIDEQ ? LONG_Q_CHUNK_BYTES : B_CHUNK_BYTES) + (p.stationary ? 0 : A_CHUNK_BYTES);
    uint8_t *smem_p = smem;
    uint8_t *smem_ring = smem + p_bytes;
    int2 *smem_staging = reinterpret_cast<int2 *>(smem_ring + (size_t)p.nstages * stage_bytes);
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(smem_ring + (size_t)p.nstages * stage_bytes + STAGING_BYTES);

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.nstages; ++s) { mbar_init(smem_u32(&ctrl->full[s]), 1); mbar_init(smem_u32(&ctrl->empty[s]), 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctrl->pfull[b]), 1);
            mbar_init(smem_u32(&ctrl->pempty[b]), p.epi_release ? 2 : 1);   // one commit per issuing warp
            mbar_init(smem_u32(&ctrl->tfull[b]), TWO_TILE ? 2 : 1);      // split issue: one commit per issuing warp
            mbar_init(smem_u32(&ctrl->tempty[b]), TWO_TILE ? EW / 2 : EW);
        }
        mbar_init(smem_u32(&ctrl->drain[0]), 1);
        mbar_init(smem_u32(&ctrl->drain[1]), 1);
        ctrl->abort = 0;
        fence_mbar_init();
        prefetch_tensormap(&mapP);
        prefetch_tensormap(&mapQ);
    }
    if (warp == 2) {
        tmem_alloc(smem_u32(&ctrl->tmem_base), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------- TMA producer
        // The whole warp walks the loop converged; one elected lane issues the copies.
        uint32_t stage = 0, phase = 0, pbuf = 0, pphase = 0;
        bool ok = true;
        Unit un;
        for (int u = 0; ok && get_unit<GROUPED, TN>(p, u, un); ++u) {
            if (un.q1 <= un.q0) continue;            // nothing for this CTA in this wave (all roles skip it)
            const int p_row = GROUPED ? un.prow0 : un.pb * P_ROWS;
            if (p.stationary) {
                ok = wait_bar_warp(&ctrl->pempty[pbuf], pphase ^ 1, ctrl, p.status, 1);
                if (!ok) break;
                if (elect_one()) {
                    const uint32_t bar = smem_u32(&ctrl->pfull[pbuf]);
                    mbar_arrive_expect_tx(bar, (uint32_t)(p.kc * A_CHUNK_BYTES));
                    for (int c = 0; c < p.kc; ++c)
                        tma_load_2d(smem_u32(smem_p + (size_t)(pbuf * p.kc + c) * A_CHUNK_BYTES), &mapP, bar,
                                    c * p.elems_per_chunk, p_row);
                }
                __syncwarp();
                if (++pbuf == (uint32_t)p_bufs(GROUPED, kc)) { pbuf = 0; pphase ^= 1; }
            }
            for (int k = 0; ok && k < un.q1 - un.q0; ++k) {
                const int q_row = (GROUPED ? un.qrow0 : 0) + tile_at<ALIGNED>(un, k) * TN;
                for (int c = 0; c < p.kc; ++c) {
                    ok = wait_bar_warp(&ctrl->empty[stage], phase ^ 1, ctrl, p.status, 2);
                    if (!ok) break;
                    if (elect_one()) {
                        const uint32_t bar = smem_u32(&ctrl->full[stage]);
                        uint8_t *sb = smem_ring + (size_t)stage * stage_bytes;
                        mbar_arrive_expect_tx(bar, (uint32_t)stage_bytes);
                        tma_load_2d(smem_u32(sb), &mapQ, bar, c * p.elems_per_chunk, q_row);
                        if (!p.stationary)
                            tma_load_2d(smem_u32(sb + (TN == LONG_TN ? LONG_Q_CHUNK_BYTES : B_CHUNK_BYTES)), &mapP, bar, c * p.elems_per_chunk, p_row);
                    }
                    __syncwarp();
                    if (++stage == (uint32_t)p.nstages) { stage = 0; phase ^= 1; }
                }
            }
        }
        if (!ok && lane == 0) {
            // aborting: shared memory may be released only after the copies already in flight have landed.  Stage s was
            // last armed in this trip round the ring (s < stage) or in the previous one; a `full` barrier that was never
            // armed reads as complete for the previous trip's parity.  Every wait is bounded (~1 ms each).
            const long long lim = 2000000LL;
            for (uint32_t s = 0; s < (uint32_t)p.nstages; ++s) {
                const uint32_t par = s < stage ? phase : phase ^ 1u;
                const long long t0 = clock64();
                while (!mbar_try_wait(smem_u32(&ctrl->full[s]), par) && clock64() - t0 < lim) {}
            }
            if (p.stationary) {
                const uint32_t nb = (uint32_t)p_bufs(GROUPED, kc);
                for (uint32_t b = 0; b < nb; ++b) {
                    const uint32_t par = b < pbuf ? pphase : pphase ^ 1u;
                    const long long t0 = clock64();
                    while (!mbar_try_wait(smem_u32(&ctrl->pfull[b]), par) && clock64() - t0 < lim) {}
                }
            }
        }
        __syncwarp();
    } else if (warp == 1 || warp == 3) {
        // -------------------------------------------------------------- MMA issuers
        // Issuing is the serial bottleneck of a short-K tile: measured on B200, a tcgen05.mma takes
        // ~70 cycles to issue, a tcgen05.commit ~70 and every mbarrier wait ~120 even when it is
        // already complete -- more than the 512 cycles the tensor core needs for the tile.  So two
        // warps issue: warp 1 owns the even tiles and accumulator 0, warp 3 the odd tiles and
        // accumulator 1; both walk the same tile sequence and skip each other's ring stages.
        // One tcgen05.commit per tile: when a whole tile's chunks fit in the ring twice over, its
        // stages are handed back to the producer by the epilogue once it has seen that commit.
        // Two issuers are only safe when consecutive tiles never share a ring stage (nstages >= 2*kc,
        // the same condition as the epilogue hand-back): otherwise the second issuer would wait on a
        // barrier that is still one phase behind, and a parity wait cannot tell phases two apart.
        // In that case warp 1 issues every tile and warp 3 stays out.
        const bool fast = p.stationary && p.epi_release && p.last_ksteps == 4;
        constexpr bool OB = KIND == KIND_STORE || KIND == KIND_SIGN;
        if constexpr (LONGK) {
            if (warp == 1) mma_issuer_long<DT, GROUPED>(p, ctrl, smem_ring, tmem_base, lane);
        } else if constexpr (TWO_TILE) {
            // (the host launches these instantiations only where the fast path's conditions hold)
            static_assert(KC == 1 || KC == 2, "alternate-tile epilogue: rows of one or two chunks");
            mma_issuer_role<DT, KC, GROUPED, OB, false, LASTK, true>(p, ctrl, smem_p, smem_ring, stage_bytes, tmem_base, warp, lane);
        } else if (fast && p.kc == 1 && !WIDEQ) mma_issuer_role<DT, 1, GROUPED, OB, false, KC == 1 ? LASTK : 4>(p, ctrl, smem_p, smem_ring, stage_bytes, tmem_base, warp, lane);
        else if (fast && p.kc == 2 && !WIDEQ) mma_issuer_role<DT, 2, GROUPED, OB, false, KC == 2 ? LASTK : 4>(p, ctrl, smem_p, smem_ring, stage_bytes, tmem_base, warp, lane);
        else mma_issuer_role<DT, 0, GROUPED, OB, WIDEQ>(p, ctrl, smem_p, smem_ring, stage_bytes, tmem_base, warp, lane);
    } else if (warp >= EPI_WARP0) {
        // ------------------------------------------------------------------ epilogue
        const int quarter = warp & 3;               // TMEM lane quarter this warp may read
        const int half = ((warp - EPI_WARP0) >> 2) & 1;   // which of the tile's two P blocks (accumulator columns half * TILE_N ..)
        const int group = (warp - EPI_WARP0) >> 3;        // 16 warps: which half of a 128-column pass, or (TWO_TILE) which tiles
        const int coff = TWO_TILE ? 0 : group * ECOLS;    // first column of this warp within a 128-column pass
        const int row_in_tile = half * TILE_M + quarter * 32 + lane;
        uint32_t acc = TWO_TILE ? group : 0, accphase = 0;
        uint32_t rstage = TWO_TILE ? group * p.kc : 0;    // next ring stage to hand back
        uint32_t tile_parity = 0;                         // TWO_TILE: parity of the number of tiles before this unit
        // candidates of a filter are decided from their rows at flush time
        constexpr int VERIFY = (DT == DT_I8 && KIND == KIND_COS) ? VERIFY_COS_I8
                               : L2_FILTER                      ? VERIFY_L2_BF16
                               : !IPCOS_FILTER                  ? VERIFY_NONE
                               : KIND == KIND_IP                ? VERIFY_IP_BF16
                                                                : VERIFY_COS_BF16;
        int2 *stage_buf = smem_staging + (warp - EPI_WARP0) * (warp_stage_bytes(EW) / 8);
        uint32_t *colterm = reinterpret_cast<uint32_t *>(stage_buf + SPAIRS);
        int stage_fill = 0;
        bool ok = true;
        Unit un;
        for (int u = 0; ok && get_unit<GROUPED, TN>(p, u, un); ++u) {
            if (un.q1 <= un.q0) continue;
            const long long i = GROUPED ? (long long)un.prow0 + row_in_tile : (long long)un.pb * P_ROWS + row_in_tile;
            const bool row_ok = GROUPED ? row_in_tile < un.prows : i < p.n;
            const bool two_blocks = GROUPED ? un.prows > TILE_M : (long long)un.pb * P_ROWS + TILE_M < p.n;
            const long long q_base = GROUPED ? un.qrow0 : 0;                          // Q row of tile 0
            const long long q_end = GROUPED ? (long long)un.qrow0 + un.qrows : p.m;   // end of the Q rows of this unit
            int ri = 0;          // I8/L2: |x|^2 - floor(r^2)
            float rf = 0.f;      // COS: t*|x|;  BF16/L2: (|x|^2 - r^2) / 2
            float rf_hi = 0.f;   // row-deciding cosine and Euclidean forms: the same with the raised threshold
            if (row_ok) {
                if constexpr (DT == DT_I8 && KIND == KIND_L2) ri = reinterpret_cast<const int *>(p.nx)[i] - p.thr_i;
                if constexpr (DT == DT_BF16 && KIND == KIND_COS) {
                    // s >= (t |x|) |y|, read off the sign of s - b like the other bf16 kinds.  The cosine with a zero
                    // vector counts as 0 (passes iff t <= 0), and the stored norms make the products say so:
                    //   t > 0: the pre-pass stores +inf for a zero vector, so b = +inf and nothing passes (a row
                    //          term that underflows to 0 becomes the smallest denormal: 0 * inf would be NaN);
                    //   t <= 0 (a zero t is passed as -0): b = -0 whenever a zero vector is involved, and
                    //          s - (-0) = +0 for a score of either zero.
                    rf = p.thr_f * reinterpret_cast<const float *>(p.nx)[i];
                    if (p.thr_f > 0.f && rf == 0.f) rf = 1.401298464e-45f;
                    if constexpr (IPCOS_FILTER) {
                        rf_hi = p.thr_hi * reinterpret_cast<const float *>(p.nx)[i];
                        if (p.thr_hi > 0.f && rf_hi == 0.f) rf_hi = 1.401298464e-45f;
                    }
                }
                if constexpr (DT == DT_I8 && KIND == KIND_COS) {
                    // fp32 filter for s >= t |x| |y|, lowered by 2^-18 relative (the fp32 roundings of t, the two norms,
                    // the products and of s itself add up to under 2^-21): a necessary condition of the exact test,
                    // which decides the surviving candidates when they leave the CTA.  t > 0: the norm of a zero
                    // vector is stored as +inf, so that nothing involving it becomes a candidate.
                    const float b = p.thr_f * reinterpret_cast<const float *>(p.nx)[i];
                    rf = b >= 0.f ? b * (1.f - 0x1p-18f) : b * (1.f + 0x1p-18f);
                }
                // BF16/L2 decides |x|^2 + |y|^2 - 2s <= r^2 as  s >= (|x|^2 - r^2)/2 + |y|^2/2:  one add per element
                if constexpr (DT == DT_BF16 && KIND == KIND_L2) {
                    if constexpr (L2_FILTER) {
                        rf = 0.5f * (reinterpret_cast<const float *>(p.nx)[i] * p.l2_xscale - p.l2_thr_filter);
                        rf_hi = 0.5f * (reinterpret_cast<const float *>(p.nx)[i] * p.l2_xscale_hi - p.l2_thr_sure);
                    }
                    else rf = 0.5f * (reinterpret_cast<const float *>(p.nx)[i] - p.thr_f);
                }
            }
            const int k_first = TWO_TILE ? (int)((group ^ tile_parity) & 1u) : 0;
            tile_parity ^= (uint32_t)(un.q1 - un.q0) & 1u;
            for (int k = k_first; ok && k < un.q1 - un.q0; k += TWO_TILE ? 2 : 1) {
                const int qt = tile_at<ALIGNED>(un, k);
                // per-tile filter bound: a necessary condition on max_j s_ij for row i to have any hit
                int fi = p.thr_i;
                float ff = p.thr_f;
                // (min, max) of the per-column term over the tile's rows.  Bucketed mode: the tile starts at any row, so
                // it takes the bounds of the one or two 256-row blocks it touches (wider, still necessary conditions).
                int qb0 = qt / (QSTAT_ROWS / TN), qb1 = qb0;
                if constexpr (GROUPED) {
                    const long long w0 = q_base + (long long)qt * TN;
                    const long long last = (p.m - 1) / QSTAT_ROWS;
                    qb0 = (int)(w0 / QSTAT_ROWS);
                    qb1 = (int)min((w0 + TN - 1) / QSTAT_ROWS, last);
                }
                if constexpr (DT == DT_I8 && KIND == KIND_L2) {
                    const int2 s0 = reinterpret_cast<const int2 *>(p.qstat)[qb0], s1 = reinterpret_cast<const int2 *>(p.qstat)[qb1];
                    fi = (ri + min(s0.x, s1.x) + 1) >> 1;         // 2s >= |x|^2 - R + min|y|^2
                }
                if constexpr (DT == DT_BF16 && KIND == KIND_COS) {
                    const float2 s0 = reinterpret_cast<const float2 *>(p.qstat)[qb0], s1 = reinterpret_cast<const float2 *>(p.qstat)[qb1];
                    ff = rf * (p.thr_f >= 0.f ? fminf(s0.x, s1.x) : fmaxf(s0.y, s1.y));     // s >= t|x| * min|y| (max|y| when t < 0)
                }
                if constexpr (DT == DT_I8 && KIND == KIND_COS) {
                    const float2 s0 = reinterpret_cast<const float2 *>(p.qstat)[qb0], s1 = reinterpret_cast<const float2 *>(p.qstat)[qb1];
                    // compared with the row maximum converted to fp32, as the element test converts the scores: the
                    // conversion is monotone, so the bound stays a necessary condition of that test
                    ff = rf * (p.thr_f >= 0.f ? fminf(s0.x, s1.x) : fmaxf(s0.y, s1.y));
                }
                if constexpr (DT == DT_BF16 && KIND == KIND_L2) {
                    const float2 s0 = reinterpret_cast<const float2 *>(p.qstat)[qb0], s1 = reinterpret_cast<const float2 *>(p.qstat)[qb1];
                    // s >= (|x|^2 - r^2)/2 + min|y|^2/2; the filter form rounds exactly as its element test does
                    if constexpr (L2_FILTER) ff = __fmaf_rn(p.l2_ycoef, fminf(s0.x, s1.x), rf);
                    else ff = rf + 0.5f * fminf(s0.x, s1.x);
                }
                // per-column terms of this warp's columns, 4 per lane, fetched while the tile is still
                // being multiplied so that the exact test never waits on global memory (fetching them only when a
                // candidate shows up was measured: no gain for sparse joins, 5 % slower dense ones)
                // int8 kinds fetch them only when a candidate shows up: measured -1.6 % (cosine) and -2.6 % (Euclidean) on a
                // sparse 262 144^2 join, +0.5-1 % on a dense one (the adaptive form -- prefetch while the previous tile
                // had candidates -- lost on both)
                constexpr bool LAZY_COLTERMS = DT == DT_I8;
                constexpr int CPL = ECOLS / 32;           // per-column terms per lane: 4, or 2 with 16 epilogue warps
                auto load_colterms = [&](int ps) -> uint4 {
                    const uint32_t *nyp = reinterpret_cast<const uint32_t *>(p.ny) + (q_base + (long long)qt * TN + ps * TILE_N + coff) + CPL * lane;
                    if constexpr (CPL == 2) {
                        if constexpr (GROUPED) return make_uint4(__ldg(nyp), __ldg(nyp + 1), 0u, 0u);
                        const uint2 t2 = __ldg(reinterpret_cast<const uint2 *>(nyp));
                        return make_uint4(t2.x, t2.y, 0u, 0u);
                    } else if constexpr (GROUPED)   // a bucket starts at any row: no 16-byte alignment
                        return make_uint4(__ldg(nyp), __ldg(nyp + 1), __ldg(nyp + 2), __ldg(nyp + 3));
                    else
                        return __ldg(reinterpret_cast<const uint4 *>(nyp));
                };
                uint4 yq_pass[NPASS];
#pragma unroll
                for (int ps = 0; ps < NPASS; ++ps) {
                    yq_pass[ps] = make_uint4(0, 0, 0, 0);
                    if constexpr ((KIND == KIND_COS || KIND == KIND_L2) && !LAZY_COLTERMS) yq_pass[ps] = load_colterms(ps);
                }
                ok = wait_bar_warp(&ctrl->tfull[acc], accphase, ctrl, p.status, 6);
                if (!ok) break;
                tc_fence_after();
                if (p.epi_release && (TWO_TILE ? ((warp - EPI_WARP0) & 7) == 0 : warp == EPI_WARP0)) {
                    // the tile's MMAs have retired: its ring stages are free again
                    // (straight-line for one or two chunks: this sits on the accumulator hand-back path
                    // of the whole CTA, and a loop with a run-time trip count costs ~40 cycles per tile)
                    if (p.kc == 1) {
                        if (lane == 0) mbar_arrive(smem_u32(&ctrl->empty[rstage]));
                        if (++rstage == (uint32_t)p.nstages) rstage = 0;
                    } else if (p.kc == 2) {
                        const uint32_t r2 = rstage + 1 == (uint32_t)p.nstages ? 0u : rstage + 1;
                        if (lane == 0) {
                            mbar_arrive(smem_u32(&ctrl->empty[rstage]));
                            mbar_arrive(smem_u32(&ctrl->empty[r2]));
                        }
                        rstage = r2 + 1 == (uint32_t)p.nstages ? 0u : r2 + 1;
                    } else {
                        for (int c = 0; c < p.kc; ++c) {
                            if (lane == 0) mbar_arrive(smem_u32(&ctrl->empty[rstage]));
                            if (++rstage == (uint32_t)p.nstages) rstage = 0;
                        }
                    }
                    if constexpr (TWO_TILE) {       // the other group hands back the next tile's stages (nstages >= 2 kc here)
                        rstage += (uint32_t)p.kc;
                        if (rstage >= (uint32_t)p.nstages) rstage -= (uint32_t)p.nstages;
                    }
                    __syncwarp();
                }
                if constexpr (TWO_TILE) {
                    // Dense output with the test "sign bit clear": no filter levels at all.  One funnel shift per column
                    // collects the sign bits of the lane's scores, 32 columns to a chain, which costs less than the
                    // maxima, votes and branches of the hierarchy when most blocks hold hits anyway.
                    static_assert(!LONGK && !NARROW && ECOLS == 64, "the flat test: standard geometry, 32-bit words");
                    uint32_t mask[4];
                    uint32_t m0 = 0, m1 = 0, m2 = 0, m3 = 0;
#pragma unroll 1
                    for (int ps = 0; ps < 2; ++ps) {
                        uint32_t v[ECOLS];
                        tmem_ld_words(tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * ACC_COLS + half * TILE_N + ps * ECOLS, v, std::false_type{});
                        if (ps == 1) {
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(smem_u32(&ctrl->tempty[acc]));
                        }
                        uint32_t c0 = 0, c1 = 0;            // column 32w + c -> bit 31 - c of chain w
#pragma unroll
                        for (int c = 0; c < 32; ++c) {
                            c0 = __funnelshift_l(v[c], c0, 1);
                            c1 = __funnelshift_l(v[32 + c], c1, 1);
                        }
                        c0 = row_ok ? __brev(~c0) : 0u;
                        c1 = row_ok ? __brev(~c1) : 0u;
                        if (ps == 0) { m0 = c0; m1 = c1; } else { m2 = c0; m3 = c1; }
                    }
                    mask[0] = m0; mask[1] = m1; mask[2] = m2; mask[3] = m3;
                    const long long j0 = q_base + (long long)qt * TN;
                    const long long left = q_end - j0;
                    if (left < TILE_N) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const long long lq = left - 32 * q;
                            mask[q] &= lq >= 32 ? 0xffffffffu : (lq <= 0 ? 0u : ((1u << (int)lq) - 1u));
                        }
                    }
                    emit_pairs<4, GROUPED, VERIFY, SPAIRS>(p, mask, lane, i, j0, stage_buf, stage_fill);
                    accphase ^= 1;                      // this group's one accumulator
                    continue;
                }
                if constexpr (KIND == KIND_SIGN) {
                    // lane <-> hyperplane (row of P), columns <-> points (rows of Q).  One vote per column collects the
                    // signs of this warp's 32 hyperplanes for that point; lane c keeps the words of columns c, c + 32, ...
                    // and stores them into the points' key records.
                    const long long j0 = q_base + (long long)qt * TN;
                    const int plane0 = un.pb * P_ROWS + half * TILE_M + quarter * 32;      // first hyperplane of this warp
                    const bool have = plane0 < (int)p.n && (half == 0 || two_blocks);
                    uint32_t v[TILE_N];
                    if (have) tmem_ld_words(tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * ACC_COLS + half * TILE_N, v, std::false_type{});
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctrl->tempty[acc]));
                    if (have) {
                        uint32_t keep[TILE_N / 32] = {0u, 0u, 0u, 0u};
#pragma unroll
                        for (int c = 0; c < TILE_N; ++c) {
                            const bool pos = DT == DT_I8 ? (int)v[c] > 0 : __uint_as_float(v[c]) > 0.f;
                            const uint32_t word = __ballot_sync(0xffffffffu, pos);
                            if ((c & 31) == lane) keep[c >> 5] = word;
                        }
#pragma unroll
                        for (int q = 0; q < TILE_N / 32; ++q) {
                            const long long j = j0 + 32 * q + lane;
                            if (j < q_end) p.key_out[j * p.key_ld + (plane0 >> 5)] = keep[q];
                        }
                    }
                    acc ^= 1;
                    if (acc == 0) accphase ^= 1;
                    continue;
                }
                if constexpr (KIND == KIND_STORE) {
                    // lane <-> row of P (an output coordinate), columns <-> rows of Q (output rows).  With two P
                    // blocks in the tile this warp stores block `half`; with one, the two warps of a lane quarter
                    // split that block's 128 columns between them.
                    const long long j0 = q_base + (long long)qt * TN;
                    uint16_t *sb = reinterpret_cast<uint16_t *>(stage_buf);          // [32 output rows][32 coordinates]
                    const int i_unit = (GROUPED ? un.prow0 : un.pb * P_ROWS) + quarter * 32;
                    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * ACC_COLS;
                    if constexpr (WIDEQ)        // one block, 256 streamed rows: this warp stores rows half * 128 ..
                        store_tile_part<TILE_N>(p, t_lane + half * TILE_N, &ctrl->tempty[acc], lane, sb, j0 + half * TILE_N, q_end, i_unit);
                    else if (two_blocks)
                        store_tile_part<TILE_N>(p, t_lane + half * TILE_N, &ctrl->tempty[acc], lane, sb, j0, q_end, i_unit + half * TILE_M);
                    else
                        store_tile_part<TILE_N / 2>(p, t_lane + half * (TILE_N / 2), &ctrl->tempty[acc], lane, sb, j0 + half * (TILE_N / 2), q_end, i_unit);
                    acc ^= 1;
                    if (acc == 0) accphase ^= 1;
                    continue;
                }
                // this warp's 128 columns of the tile (long rows: two passes of 128 over its block's 256), then hand
                // the accumulator back to the MMA warp
                constexpr int NV = NARROW ? ECOLS / 2 : ECOLS;            // accumulator words per thread
                constexpr int GCOLS = 16, NG = ECOLS / GCOLS, GW = NV / NG;     // column groups of level 1
                constexpr uint32_t GMASK = (1u << GCOLS) - 1u;
                constexpr int MODE = DT == DT_BF16 ? MAX_F32 : (NARROW ? MAX_S16X2 : MAX_S32);
                // Long rows with the packed epilogue: both passes' words fit in registers (2 x 64), so the single
                // accumulator goes back to the MMA warp before any test runs instead of after the first pass's.
                constexpr bool LOAD_ALL = LONGK && NARROW;
                uint32_t vall[LOAD_ALL ? NPASS : 1][NV];
                if constexpr (LOAD_ALL) {
#pragma unroll
                    for (int ps = 0; ps < NPASS; ++ps)
                        tmem_ld_words(tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * ACC_COLS + half * TN + ps * TILE_N + coff, vall[ps],
                                      std::integral_constant<bool, NARROW>{});
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctrl->tempty[acc]));
                }
#pragma unroll
                for (int ps = 0; ps < NPASS; ++ps) {
                uint4 yq = yq_pass[ps];
                uint32_t (&v)[NV] = vall[LOAD_ALL ? ps : 0];
                if constexpr (!LOAD_ALL) {
                    tmem_ld_words(tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * ACC_COLS + half * TN + ps * TILE_N + coff, v,
                                  std::integral_constant<bool, NARROW>{});
                    tc_fence_before();
                    __syncwarp();
                    if (ps == NPASS - 1 && lane == 0) mbar_arrive(smem_u32(&ctrl->tempty[acc]));
                }
                // level 0: the row maximum over this warp's 128 columns against the per-tile bound
                // (a necessary condition of the exact test, in the same arithmetic)
                auto bound_ok = [&](uint32_t word) -> bool {
                    if constexpr (DT == DT_I8) {
                        const int mx = NARROW ? max((int)(short)(word & 0xffffu), (int)word >> 16) : (int)word;
                        if constexpr (KIND == KIND_COS) return (float)mx >= ff;
                        return mx >= fi;
                    } else {
                        return __uint_as_float(word) >= ff;
                    }
                };
                // bf16: taken over the maxima of the 16-column groups, which level 1 then has for free (dense
                // outputs: -6 %); int8 keeps one flat tree, measured 5 % faster on the sparse headline join
                constexpr bool GROUP_FIRST = DT == DT_BF16;
                uint32_t gmax[NG];
                bool hit;
                if constexpr (GROUP_FIRST) {
#pragma unroll
                    for (int k = 0; k < NG; ++k) gmax[k] = TreeMax<GW, MODE>::run(v + k * GW);
                    hit = row_ok && bound_ok(TreeMax<NG, MODE>::run(gmax));
                } else {
                    hit = row_ok && bound_ok(TreeMax<NV, MODE>::run(v));
                }
                if (__builtin_expect(__any_sync(0xffffffffu, hit) != 0, 0)) {   // rare for sparse joins: keep it out of line
                    // level 1: which 16-column groups can hold a hit for this row
                    uint32_t gm = 0;
#pragma unroll
                    for (int k = 0; k < NG; ++k) {
                        if constexpr (!GROUP_FIRST) gmax[k] = TreeMax<GW, MODE>::run(v + k * GW);
                        gm |= (bound_ok(gmax[k]) ? 1u : 0u) << k;
                    }
                    if (!row_ok) gm = 0;
                    const long long j0 = q_base + (long long)qt * TN + ps * TILE_N + coff;
                    uint32_t mask[ECOLS / 32];
                    uint32_t cand[ECOLS / 32];          // row-deciding forms: passing columns that are not sure to pass
#pragma unroll
                    for (int q = 0; q < ECOLS / 32; ++q) mask[q] = cand[q] = 0;
                    if constexpr (KIND != KIND_IP) {
                        // the per-column terms go through shared memory: level 2 reads 16 of them per group as four
                        // broadcast loads (a shuffle per term cost four times the instructions)
                        if constexpr (LAZY_COLTERMS) yq = load_colterms(ps);
                        __syncwarp();
                        if constexpr (CPL == 2) reinterpret_cast<uint2 *>(colterm)[lane] = make_uint2(yq.x, yq.y);
                        else reinterpret_cast<uint4 *>(colterm)[lane] = yq;
                        __syncwarp();
                    }
#pragma unroll
                    for (int k = 0; k < NG; ++k) {
                        if (!__any_sync(0xffffffffu, (gm >> k) & 1u)) continue;
                        // level 2: the exact test on the 16 columns of group k
                        uint32_t yw[GCOLS];                                     // per-column term of Q (norm kinds)
                        if constexpr (KIND != KIND_IP) {
#pragma unroll
                            for (int t = 0; t < GCOLS / 4; ++t) {
                                const uint4 q4 = reinterpret_cast<const uint4 *>(colterm)[k * (GCOLS / 4) + t];
                                yw[4 * t] = q4.x;
                                yw[4 * t + 1] = q4.y;
                                yw[4 * t + 2] = q4.z;
                                yw[4 * t + 3] = q4.w;
                            }
                        }
                        uint32_t mk = 0;
                        if constexpr (DT == DT_BF16) {
                            // The same decision as bound_ok, taken from a sign bit: fl(s - b) >= +0 exactly when
                            // s >= b.  The adds run on the FMA pipe and one funnel shift collects the bit, where a
                            // compare, a select and an OR would all queue on the half-rate ALU pipe (dense outputs).
                            // Four independent chains of four columns.
                            constexpr int NCH = GCOLS / 4;
                            uint32_t fail[NCH];
#pragma unroll
                            for (int q = 0; q < NCH; ++q) fail[q] = 0;
#pragma unroll
                            for (int c = 0; c < GCOLS; ++c) {
                                const float b = KIND == KIND_IP    ? p.thr_f
                                                : KIND == KIND_COS ? __fmul_rn(rf, __uint_as_float(yw[c]))   // as level 0 rounds it
                                                : L2_FILTER        ? __fmaf_rn(p.l2_ycoef, __uint_as_float(yw[c]), rf)
                                                                   : rf + 0.5f * __uint_as_float(yw[c]);
                                fail[c >> 2] = __funnelshift_l(__float_as_uint(__uint_as_float(v[k * GCOLS + c]) - b), fail[c >> 2], 1);
                            }
                            // chain q holds columns 4q .. 4q+3 at bits 3 .. 0
                            uint32_t fall = 0;                                  // column c -> bit GCOLS - 1 - c
#pragma unroll
                            for (int q = 0; q < NCH; ++q) fall |= fail[q] << (4 * (NCH - 1 - q));
                            mk = (__brev(~fall) >> (32 - GCOLS)) & GMASK;
                            if constexpr (IPCOS_FILTER || L2_FILTER) {
                                // sure to pass: s > b_hi, the sign bit of fl(b_hi - s) (a score equal to the bound stays a candidate)
                                uint32_t sure[NCH];
#pragma unroll
                                for (int q = 0; q < NCH; ++q) sure[q] = 0;
#pragma unroll
                                for (int c = 0; c < GCOLS; ++c) {
                                    const float bh = KIND == KIND_IP    ? p.thr_hi
                                                     : KIND == KIND_COS ? __fmul_rn(rf_hi, __uint_as_float(yw[c]))
                                                                        : __fmaf_rn(p.l2_ycoef_hi, __uint_as_float(yw[c]), rf_hi);
                                    sure[c >> 2] = __funnelshift_l(__float_as_uint(bh - __uint_as_float(v[k * GCOLS + c])), sure[c >> 2], 1);
                                }
                                uint32_t sall = 0;
#pragma unroll
                                for (int q = 0; q < NCH; ++q) sall |= sure[q] << (4 * (NCH - 1 - q));
                                const uint32_t mk_cand = mk & ~((__brev(sall) >> (32 - GCOLS)) & GMASK);
                                if ((gm >> k) & 1u) cand[(k * GCOLS) >> 5] |= mk_cand << ((k * GCOLS) & 31);
                            }
                        } else {
#pragma unroll
                        for (int c = 0; c < GCOLS; ++c) {
                            uint32_t x;
                            if constexpr (NARROW) {
                                const uint32_t w = v[(k * GCOLS + c) >> 1];
                                x = (c & 1) ? (uint32_t)((int)w >> 16) : (uint32_t)(int)(short)(w & 0xffffu);
                            } else {
                                x = v[k * GCOLS + c];
                            }
                            bool pass = false;
                            if constexpr (DT == DT_I8 && KIND == KIND_IP) pass = (int)x >= p.thr_i;
                            if constexpr (DT == DT_I8 && KIND == KIND_L2) pass = 2 * (int)x - (int)yw[c] >= ri;
                            if constexpr (DT == DT_I8 && KIND == KIND_COS) pass = (float)(int)x >= rf * __uint_as_float(yw[c]);
                            mk |= (pass ? 1u : 0u) << c;
                        }
                        }
                        if (!((gm >> k) & 1u)) mk = 0;       // the group bound is necessary: nothing can pass here
                        mask[(k * GCOLS) >> 5] |= mk << ((k * GCOLS) & 31);
                    }
                    // columns past the end of Q (of the bucket) were multiplied as zero rows: drop them
                    const long long left = q_end - j0;
                    if (left < ECOLS) {
#pragma unroll
                        for (int q = 0; q < ECOLS / 32; ++q) {
                            const long long lq = left - 32 * q;
                            mask[q] &= lq >= 32 ? 0xffffffffu : (lq <= 0 ? 0u : ((1u << (int)lq) - 1u));
                        }
                    }
                    emit_pairs<ECOLS / 32, GROUPED, VERIFY, SPAIRS>(p, mask, lane, i, j0, stage_buf, stage_fill, cand);
                }
                }   // passes
                if constexpr (LONGK) {
                    accphase ^= 1;                      // one accumulator buffer
                } else {
                    acc ^= 1;
                    if (acc == 0) accphase ^= 1;
                }
            }
        }
        if (ok) flush_pairs<GROUPED, VERIFY>(p, stage_buf, stage_fill, lane);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 2) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
    if (p.host_result != nullptr && threadIdx.x == 0) {
        // every pair of this CTA has been counted (the epilogue warps flushed before the barrier above)
        __threadfence();
        if (atomicAdd(p.done_ticket, 1u) == gridDim.x - 1) {
            __threadfence();
            p.host_result[0] = atomicAdd(p.counter, 0ull);
            p.host_result[1] = (unsigned long long)atomicOr(p.status, 0u);
            __threadfence_system();
        }
    }
}

// Self-test of the bounded wait: one warp waits on a barrier that nothing ever completes, with a
// short cycle budget.  The wait must give up, raise the status word and let the kernel return.
__global__ void wait_timeout_selftest_kernel(unsigned int *status, long long limit_cycles) {
    __shared__ Ctrl ctrl;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&ctrl.full[0]), 1);
        ctrl.abort = 0;
        fence_mbar_init();
    }
    __syncthreads();
    const bool ok = wait_bar(&ctrl.full[0], 0, &ctrl, status, 0x7f, limit_cycles);
    if (ok && threadIdx.x == 0) atomicCAS(status, 0u, 0x40000000u);   // must not happen: flags a false wake-up
}

}  // namespace sj
