// Fused path: ONE launch per evicting step.  A thread-block cluster of C CTAs owns one unit
// (one KV head of one layer of one sequence) from the anchor to the compacted K and V, and goes
// on to the next unit (u + number of clusters) with the next unit's K rows already on their way:
//
//   load K      every CTA pulls its contiguous slice of the unit's n key rows on chip exactly
//               once: most rows into shared memory with TMA bulk copies (cp.async.bulk, one
//               mbarrier per 16-row tile), the remainder into registers with 128-bit loads.
//               Nothing is read from HBM twice.
//   anchor      (App. B.1, expr. 1)  one-pass steps: the sum of the terms k/||k|| over the cached
//               rows is carried from step to step (running sum + every CTA's delta of the last
//               step, folded in double); only the B block rows are normalised, C-th part per CTA,
//               the shares meet in every CTA's table through DSMEM stores.  Two-pass steps (first
//               evicting step, after appends, on request) sum all n rows instead.
//   scores      (App. B.1, expr. 2)  e_i = -(mu.k_i)/max(||mu|| ||k_i||, eps) from the on-chip
//               rows, norm and dot product in one pass; the orderable key of e_i goes into this
//               CTA's part of the key table, and the part is pushed to every peer with one bulk
//               copy each (shared::cluster destination), counted on the peer's own mbarrier: a CTA
//               selects as soon as ITS table is complete, without a cluster barrier.  fp32 scores
//               go to global scratch, coalesced.
//   select      every CTA selects on its own copy of the table.  Only E = n - N keys go, so the
//               work is at the low end: a 2048-bin histogram over the unit's own key range, the bin
//               where the running count from below reaches E, a bitmap of the tokens under that
//               bin, an exact rank among the bin's own few keys.  Crowded bins (many equal scores)
//               fall back to a histogram over a fixed-point image of e with an exact rank or a
//               4x8-bit radix select.  Ties keep the older token (Eq. efficient-keydiff, topk).
//   compact     prefix counts over the bitmap give every kept row its destination; the rows then
//               leave the chip tile by tile, and each shared-memory tile is refilled as soon as
//               it has been written out: K stores hand their tile to the V load of the same rows,
//               V stores hand it to the K load of the cluster's next unit, which the owning warp
//               scores while the following tile's stores drain (Eq. keydiff, in place, token
//               order).  The evicted rows' terms are taken off the running sum on the way out.
//
// Cluster barriers per unit: ONE (before the V stores; two-pass steps have a second, for the anchor's
// partial sums).  In-place safety: a CTA's K stores start
// after its key table is complete, i.e. after every peer has scored -- hence holds on chip -- all
// its K rows of the unit.  Every warp arrives at the cluster barrier only after the V rows it is
// responsible for have landed (bulk copies waited for, register loads consumed), and no V store is
// issued before that barrier's wait: every V row that moves is then on chip.
//
// No multicast TMA is used anywhere; each CTA issues its own bulk loads.  Every mbarrier wait is
// bounded: on expiry the kernel records KEYDIFF_ERR_TIMEOUT in the status word and carries on
// to its normal exit (all CTAs still meet at every cluster barrier).
#pragma once
#include "common.cuh"
#include "select.cuh"
#include "staged_kernels.cuh"   // concat_row

namespace kd {

constexpr int kFusedThreads = 512;
constexpr int kFusedWarps = kFusedThreads / 32;
constexpr int kGroups = kFusedThreads / kLanesPerRow;   // 64 row groups per CTA
constexpr int kTileRows = 16;                           // one bulk copy = one tile of 16 rows (4 KB)
constexpr int kMaxTiles = 52;                           // <= 832 rows of a slice live in shared memory
constexpr int kTilesPerWarp = (kMaxTiles + kFusedWarps - 1) / kFusedWarps;
constexpr int kMaxRegRows = 6;                          // + up to 6 rows per group (384 rows) in registers
constexpr int kBins = 2048;                             // histogram over e in [-1, 1]
constexpr int kCandCap = kFusedThreads;                 // exact-rank stage handles this many candidates
constexpr int kMaxCluster = 16;
constexpr int kFastKeys = 17;                           // fast select: keys per thread held in registers (n <= 8704)
constexpr int kFastCandCap = 192;                       // fast select: keys of the threshold bin ranked exactly
constexpr int kReduceBytes = 16 * 1024;   // least size of the key-table region: while the table is dead it lends two [8][128] double tables
constexpr int kSmemLimit = 232448;                      // opt-in shared memory per CTA on sm_100
constexpr int kErrTimeout = -6;                         // KEYDIFF_ERR_TIMEOUT
constexpr uint32_t kWaitSpins = 1u << 24;               // bound of every mbarrier wait

struct FusedLayout {
    int rows, keys, work, xchg, bitmap, sel, mu, mbar, misc, total;
};

// Shared-memory carve-up for a slice with `smem_rows` resident rows, a key table of nkeys
// entries and a cluster of C CTAs.
__host__ __device__ inline FusedLayout fused_layout(int smem_rows, int nkeys, int C) {
    FusedLayout L;
    int off = 0;
    auto take = [&off](int bytes) { const int o = off; off += (bytes + 127) & ~127; return o; };
    // the regions whose size does not depend on the launch come first: their addresses are compile-time constants, which
    // keeps them out of the registers
    L.misc = take(128);
    L.mbar = take((kMaxTiles + 1) * 8);   // one per tile + the key exchange's
    L.mu = take(2 * kHeadDim * 4);   // this unit's anchor and the next unit's
    L.sel = take(static_cast<int>(sizeof(SelectSmem)));
    L.work = take(kBins * 4);   // warp-reduction scratch / histogram / destination table (never live together)
    L.rows = take(smem_rows * kRowBytes);
    L.keys = take(nkeys * 4 > kReduceBytes ? nkeys * 4 : kReduceBytes);   // also the reduction scratch while the table is dead
    L.xchg = take(2 * kCandCap * 4 + C * kHeadDim * 8);   // candidates of the threshold bin | [C][128] doubles pushed by the peers
    L.bitmap = take(2 * ((nkeys + 31) / 32) * 4);   // evicted-token bitmap, evicted-before count of every word
    L.total = off;
    return L;
}

struct FusedParams {
    uint4* k_cache; uint4* v_cache; const uint4* new_k; const uint4* new_v;
    int len, B, N, U;
    float eps;
    int cluster;        // CTAs per cluster
    int rows_per_cta;   // slice length = ceil(n / cluster) rounded up to a multiple of 4
    int smem_rows;      // rows of a slice held in shared memory (multiple of kTileRows)
    int nkeys;          // key-table capacity (>= cluster * rows_per_cta)
    int nmax;           // row stride of the score scratch
    unsigned stagger_ns; // cluster c starts c * stagger_ns late (see the kernel)
    float* scores; int32_t* kept_idx; int32_t* first_evicted;
    unsigned long long* moved_rows; int32_t* status;
    // running anchor (see the kernel): sum of k/||k|| over the cached rows as of the previous step
    // = anchor_in[u][c] + sum over CTA ranks r of anchor_delta[u][r][c]; this step writes anchor_out and
    // new deltas
    const double* anchor_in; double* anchor_out; double* anchor_delta;
    int raw_anchor;     // 1: the anchor is the mean of the keys themselves (Sec. 3.2), 0: of the normalised keys
    int window;         // w most recent tokens that are never evicted (Sec. 3.2, sliding window)
    int32_t* kept_mirror;   // optional second destination of the kept-index list (device alias of pinned host memory)
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ uint32_t cluster_ctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_sync_all() { cluster_arrive(); cluster_wait(); }
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r; asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank)); return r;
}
__device__ __forceinline__ void st_cluster_v4(uint32_t addr, const uint4& v) {
    asm volatile("st.shared::cluster.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// global -> this CTA's shared memory, completion counted on an mbarrier; 16-byte aligned, size % 16 == 0
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// this CTA's shared memory -> a peer CTA's shared memory (cluster addresses of the destination and of the PEER's
// mbarrier, which counts the bytes as they land); 16-byte aligned, size % 16 == 0.  A plain peer-to-peer copy inside
// the cluster: no multicast.
__device__ __forceinline__ void bulk_push(uint32_t dst_cluster, uint32_t src, uint32_t bytes, uint32_t bar_cluster) {
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_cluster), "r"(src), "r"(bytes), "r"(bar_cluster) : "memory");
}
// orders this thread's earlier shared-memory writes in front of later reads of them by the copy engine
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t;
}

// Optional per-phase timing (build with -DKEYDIFF_PHASE_STAMPS, see build.py --phase-stamps): thread 0 of every CTA
// adds the time since its previous stamp to the phase's total; at the end of the kernel the totals go to
// g_phase_ns[CTA][phase], which keydiff_debug_phase_ns reads.  Without the macro nothing of this is compiled.
constexpr int kMaxPhases = 16;
constexpr int kMaxStampCtas = 2368;   // 148 SMs x 16
#ifdef KEYDIFF_PHASE_STAMPS
__device__ unsigned long long g_phase_ns[kMaxStampCtas][kMaxPhases];
#define KD_STAMP_DECL __shared__ unsigned long long stamp_sh[kMaxPhases + 1]; \
    if (threadIdx.x == 0) { for (int i_ = 0; i_ < kMaxPhases; ++i_) stamp_sh[i_] = 0; stamp_sh[kMaxPhases] = global_timer_ns(); }
#define KD_STAMP(id) do { if (threadIdx.x == 0) { const unsigned long long now_ = global_timer_ns(); \
    stamp_sh[id] += now_ - stamp_sh[kMaxPhases]; stamp_sh[kMaxPhases] = now_; } } while (0)
#define KD_STAMP_FLUSH do { if (threadIdx.x == 0 && blockIdx.x < kMaxStampCtas) \
    for (int i_ = 0; i_ < kMaxPhases; ++i_) atomicAdd(&g_phase_ns[blockIdx.x][i_], stamp_sh[i_]); } while (0)
#else
#define KD_STAMP_DECL
#define KD_STAMP(id) do {} while (0)
#define KD_STAMP_FLUSH do {} while (0)
#endif

// Bounded wait; returns false if the phase never completed.  The first wait that runs out records
// KEYDIFF_ERR_TIMEOUT in the status word; while the status word is non-zero every other wait gives up after
// a thousand polls instead of waiting its full length again, so a kernel in which one copy never lands still
// ends within milliseconds.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int32_t* status, uint32_t limit = kWaitSpins) {
    for (uint32_t spin = 0; spin < limit; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 1023u) == 1023u && *reinterpret_cast<volatile int32_t*>(status) != 0) return false;
    }
    atomicExch(status, kErrTimeout);
    return false;
}

// Failure-detection self test: every thread waits, with a limit of `polls` polls, on an mbarrier that nothing
// ever completes (no arrival, no copy).  The waits run out, the status word receives KEYDIFF_ERR_TIMEOUT and
// the kernel returns normally: exactly what a product kernel does when a copy never lands.
__global__ void bounded_wait_selftest_kernel(int32_t* status, uint32_t polls) {
    __shared__ __align__(8) unsigned long long bar;
    const uint32_t bar_sa = smem_addr(&bar);
    if (threadIdx.x == 0) {
        mbar_init(bar_sa, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    mbar_wait(bar_sa, 0u, status, polls);   // phase 0 never completes
}

// inverse of order_key
__device__ __forceinline__ float key_score(uint32_t key) {
    return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}
// Histogram bin of an orderable key: e in [-1, 1] is shifted into the single binade [2, 4), where
// the fp32 mantissa is a fixed-point image of the value; its top 11 bits are 2048 equal bins.  The
// map is monotone non-decreasing in e (rounding and clamping are), which is all selection needs.
__device__ __forceinline__ int key_bin(uint32_t key) {
    const float f = fmaxf(fminf(key_score(key) + 3.0f, 3.9999998f), 2.0f);
    return static_cast<int>((__float_as_uint(f) >> 12) & (kBins - 1));
}

// Geometry of one CTA's slice of a unit (identical for every unit of a step).
struct Slice {
    int seg_a, seg;     // first unit row, number of rows
    int rs;             // rows resident in shared memory (the first rs of the slice)
    int ntiles;         // ceil(rs / kTileRows)
};

// One thread: start the bulk load of tile `tile` (local rows [16*tile, min(rs, 16*tile+16))) of unit
// u's slice on that tile's mbarrier.  Rows below `len` come from the cache tensor, the rest from
// the block tensor.
__device__ __forceinline__ void issue_tile(const uint4* cache, const uint4* block, int u, int len, int B, int N,
                                           const Slice& s, int tile, uint32_t rows_sa, uint32_t mbar_sa) {
    const int lo = tile * kTileRows, hi = min(s.rs, lo + kTileRows);
    const int g0 = s.seg_a + lo;                               // first unit row of the tile
    const int from_cache = min(max(len - g0, 0), hi - lo);
    const int from_block = (hi - lo) - from_cache;
    const uint32_t bar = mbar_sa + 8 * tile, dst = rows_sa + lo * kRowBytes;
    mbar_expect_tx(bar, (hi - lo) * kRowBytes);
    if (from_cache > 0)
        bulk_load(dst, cache + (static_cast<size_t>(u) * N + g0) * kRowVec, from_cache * kRowBytes, bar);
    if (from_block > 0)
        bulk_load(dst + from_cache * kRowBytes,
                  block + (static_cast<size_t>(u) * B + (g0 + from_cache - len)) * kRowVec, from_block * kRowBytes, bar);
}

// ---------------------------------------------------------------- row arithmetic (packed fp32 pairs)
// A lane's two 128-bit words of a row as 8 fp32 pairs; pair p holds channels lane_channel(t, 2p) and
// lane_channel(t, 2p + 1).
__device__ __forceinline__ void unpack_pairs(const uint4& a, const uint4& b, float2 (&x)[8]) {
    x[0] = make_float2(bf16_lo(a.x), bf16_hi(a.x)); x[1] = make_float2(bf16_lo(a.y), bf16_hi(a.y));
    x[2] = make_float2(bf16_lo(a.z), bf16_hi(a.z)); x[3] = make_float2(bf16_lo(a.w), bf16_hi(a.w));
    x[4] = make_float2(bf16_lo(b.x), bf16_hi(b.x)); x[5] = make_float2(bf16_lo(b.y), bf16_hi(b.y));
    x[6] = make_float2(bf16_lo(b.z), bf16_hi(b.z)); x[7] = make_float2(bf16_lo(b.w), bf16_hi(b.w));
}
__device__ __forceinline__ float approx_rsqrt(float v) { float r; asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v)); return r; }
__device__ __forceinline__ float approx_sqrt(float v) { float r; asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v)); return r; }
__device__ __forceinline__ float approx_rcp(float v) { float r; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v)); return r; }

// ||k||^2 over the row group (two FMA chains per lane, then the 8-lane butterfly)
__device__ __forceinline__ float pairs_sumsq(const float2 (&x)[8]) {
    float2 s0 = make_float2(0.f, 0.f), s1 = s0;
#pragma unroll
    for (int p = 0; p < 4; ++p) { s0 = __ffma2_rn(x[p], x[p], s0); s1 = __ffma2_rn(x[4 + p], x[4 + p], s1); }
    return group_sum((s0.x + s0.y) + (s1.x + s1.y));
}
// mu.k.  Products and chains of four of them are fp32: such a chain rounds at the size of a few terms, and 32
// chains with independent roundings leave about 1e-8 of the size of the terms.  Everything above the chains --
// the four chains of a lane, the eight lanes of the row group -- is added in double precision: a cosine near
// zero is a cancelling sum, and fp32 partial sums of the size of ALL its terms would decide its last digits.
__device__ __forceinline__ double lane_dot(const float2 (&x)[8], const float2 (&w)[8]) {
    float2 d0 = make_float2(0.f, 0.f), d1 = d0;
#pragma unroll
    for (int p = 0; p < 4; ++p) { d0 = __ffma2_rn(x[p], w[p], d0); d1 = __ffma2_rn(x[4 + p], w[4 + p], d1); }
    return (static_cast<double>(d0.x) + static_cast<double>(d0.y)) + (static_cast<double>(d1.x) + static_cast<double>(d1.y));
}
// This lane's 16 anchor channels as fp32 pairs: w[q] = channels lane_channel(t, 2q), lane_channel(t, 2q + 1).
__device__ __forceinline__ void load_anchor(const float* mu, int t, float2 (&w)[8]) {
#pragma unroll
    for (int q = 0; q < 8; ++q) w[q] = *reinterpret_cast<const float2*>(&mu[lane_channel(t, 2 * q)]);
}
// Step a1 for one row: returns ||k||; adds k / max(||k||, eps) into acc when the row is valid.
// 1/max(r, eps) = min(1/r, 1/eps); the reciprocal square root and the square root are the
// hardware approximations (relative error about 2^-22, far inside the score tolerance).
// raw: the anchor is the mean of the keys themselves (Sec. 3.2), so k is added as it is.
__device__ __forceinline__ float row_a1(const uint4& a, const uint4& b, bool valid, float inv_eps, float2 (&acc)[8], bool raw) {
    float2 x[8];
    unpack_pairs(a, b, x);
    const float ss = pairs_sumsq(x);
    const float inv = valid ? (raw ? 1.0f : fminf(approx_rsqrt(ss), inv_eps)) : 0.f;
    const float2 inv2 = make_float2(inv, inv);
#pragma unroll
    for (int p = 0; p < 8; ++p) acc[p] = __ffma2_rn(x[p], inv2, acc[p]);
    return approx_sqrt(ss);
}
// One lane's share of ||k||^2 (fp32: the norm only enters the score as a factor) and of mu.k (double), no
// exchange between lanes yet.
__device__ __forceinline__ void lane_sumsq_dot(const uint4& a, const uint4& b, const float2 (&w)[8], float& ss, double& dot) {
    float2 x[8];
    unpack_pairs(a, b, x);
    float2 s0 = make_float2(0.f, 0.f), s1 = s0;
#pragma unroll
    for (int p = 0; p < 4; ++p) { s0 = __ffma2_rn(x[p], x[p], s0); s1 = __ffma2_rn(x[4 + p], x[4 + p], s1); }
    ss = (s0.x + s0.y) + (s1.x + s1.y);
    dot = lane_dot(x, w);
}
// Four values per lane, each to be summed over the 8 lanes of a row group: a butterfly that halves the
// values it carries (2 + 1 + 1 exchanges instead of 4 x 3).  Lane t (0..7 within the group) returns the
// group's sum of v[t >> 1].
template <typename T>
__device__ __forceinline__ T group_sum4(const T (&v)[4], int t) {
    const bool h4 = t & 4, h2 = t & 2;
    T r2[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) r2[i] = (h4 ? v[i + 2] : v[i]) + __shfl_xor_sync(0xffffffffu, h4 ? v[i] : v[i + 2], 4);
    const T r1 = (h2 ? r2[1] : r2[0]) + __shfl_xor_sync(0xffffffffu, h2 ? r2[0] : r2[1], 2);
    return r1 + __shfl_xor_sync(0xffffffffu, r1, 1);
}
// Keys of four rows of a row group from the lanes' shares ss[i] of ||k_i||^2 and dot[i] of mu.k_i: lane t
// returns row (t >> 1)'s key.
__device__ __forceinline__ uint32_t score4(const float (&ss)[4], const double (&dot)[4], int t, float m, float eps) {
    const float r2 = group_sum4(ss, t);
    const float d = static_cast<float>(group_sum4(dot, t));
    const float e = -(d * approx_rcp(fmaxf(m * approx_sqrt(r2), eps)));
    return order_key(e == 0.f ? 0.f : e);
}
// Step a2 for one row: orderable key of e = -(mu.k)/max(||mu|| ||k||, eps), -0 mapped to +0.
__device__ __forceinline__ uint32_t row_a2(const uint4& a, const uint4& b, const float2 (&w)[8], float m, float r, float eps) {
    float2 x[8];
    unpack_pairs(a, b, x);
    const float dot = static_cast<float>(group_sum(lane_dot(x, w)));
    const float e = -(dot * approx_rcp(fmaxf(m * r, eps)));
    return order_key(e == 0.f ? 0.f : e);
}

// Sum over the CTA of every thread's 16 channel accumulators (fp32 sums over a few rows each), carried in double
// from here on: an anchor sum over thousands of unit vectors cancels when the keys point in many directions, and
// fp32 partial sums of its size would limit the anchor's accuracy (hence every score's) to about 1e-7 / ||mu||.
// Returns channel tid's sum in threads tid < 128 (0 elsewhere).  scratch: half * 8 * 128 doubles, half = 1
// (two rounds of eight warps) or 2 (one round); ends after a CTA barrier only when the caller adds one.
template <int kHalf>
__device__ __forceinline__ double cta_channel_sum(const double (&v)[16], double* scratch, int tid) {
    const int lane = tid & 31, warp = tid >> 5, t = tid & 7;
    double r[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        double x = v[j];
        x += __shfl_xor_sync(0xffffffffu, x, 8);
        x += __shfl_xor_sync(0xffffffffu, x, 16);
        r[j] = x;
    }
    double s = 0.0;
    constexpr int kWarpsPerRound = 8 * kHalf;
#pragma unroll 1
    for (int w0 = 0; w0 < kFusedWarps; w0 += kWarpsPerRound) {
        if (w0 > 0) __syncthreads();   // the previous round's values have been read
        if (lane < 8 && warp >= w0 && warp < w0 + kWarpsPerRound) {
#pragma unroll
            for (int q = 0; q < 8; ++q)
                *reinterpret_cast<double2*>(&scratch[(warp - w0) * kHeadDim + lane_channel(t, 2 * q)]) = make_double2(r[2 * q], r[2 * q + 1]);
        }
        __syncthreads();
        if (tid < kHeadDim) {
#pragma unroll
            for (int w = 0; w < kWarpsPerRound; ++w) s += scratch[w * kHeadDim + tid];
        }
    }
    return s;
}
__device__ __forceinline__ void widen_acc(const float2 (&acc)[8], double (&v)[16]) {
#pragma unroll
    for (int q = 0; q < 8; ++q) { v[2 * q] = static_cast<double>(acc[q].x); v[2 * q + 1] = static_cast<double>(acc[q].y); }
}
__device__ __forceinline__ void st_cluster_f64(uint32_t addr, double v) {
    asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(addr), "d"(v) : "memory");
}

// Search in the 2048-bin histogram from the low end, two levels and one CTA barrier: warp w sums bins
// [128w, 128w+128); every warp then finds the owner warp from the 16 totals and scans that warp's 128
// bins (4 per lane).  Returns (smallest bin whose inclusive running count reaches E) << 16 | count
// strictly below it, or -1 if the total stays under E.  All threads must call; the result is uniform.
__device__ __forceinline__ int find_crossing(const int* h, int E, int lane, int warp, int* wtot) {
    const int4 v = reinterpret_cast<const int4*>(h)[32 * warp + lane];
    int s = (v.x + v.y) + (v.z + v.w);
    s = __reduce_add_sync(0xffffffffu, s);
    if (lane == 0) wtot[warp] = s;
    __syncthreads();
    const int t = lane < kFusedWarps ? wtot[lane] : 0;
    int incl = t;
#pragma unroll
    for (int o = 1; o < 16; o <<= 1) { const int x = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += x; }
    const unsigned hit = __ballot_sync(0xffffffffu, lane < kFusedWarps && incl - t < E && E <= incl);
    if (hit == 0) return -1;
    const int W = __ffs(hit) - 1;
    const int base = __shfl_sync(0xffffffffu, incl - t, W);
    const int4 c = reinterpret_cast<const int4*>(h)[32 * W + lane];
    const int c4 = (c.x + c.y) + (c.z + c.w);
    int incl2 = c4;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int x = __shfl_up_sync(0xffffffffu, incl2, o); if (lane >= o) incl2 += x; }
    const unsigned hit2 = __ballot_sync(0xffffffffu, base + incl2 >= E);
    const int J = __ffs(hit2) - 1;          // hit2 != 0: warp W's range crosses E
    int before = base + __shfl_sync(0xffffffffu, incl2 - c4, J);
    const int cx = __shfl_sync(0xffffffffu, c.x, J), cy = __shfl_sync(0xffffffffu, c.y, J), cz = __shfl_sync(0xffffffffu, c.z, J);
    const int bin = 128 * W + 4 * J;
    if (before + cx >= E) return (bin << 16) | before;
    before += cx;
    if (before + cy >= E) return ((bin + 1) << 16) | before;
    before += cy;
    if (before + cz >= E) return ((bin + 2) << 16) | before;
    return ((bin + 3) << 16) | (before + cz);
}

// Selection at the low end of the key table (every thread of the CTA calls; the result is uniform).  Only
// E = n - N keys go, so thread t looks at the keys of tokens t, t + 512, ... only (in registers up to n = 8704); the 2048
// bins are spread over the low end of the unit's own key range, from the smallest key to a bound on the
// E-th smallest (monotone in the key, which is all selection needs); the tokens under the threshold bin go
// straight into the bitmap, the bin's own few keys are ranked exactly under (key ascending, index
// descending) = the reverse of the keep order.  On entry hist and bitmap are zero, misc[0] = 0, misc[1] = n,
// all visible to the CTA.  Returns true with the evicted tokens' bits set in `bitmap` and misc[1] = the first
// evicted token (both visible to the CTA), or false when the threshold bin holds more than kFastCandCap
// keys (many equal scores): the bitmap and misc are then in an unspecified state and the caller takes the
// full-table route.  cand_key / cand_idx: kFastCandCap entries each.
// kInRegs: the thread's keys stay in registers between the passes (n <= 8704); otherwise they are read again from
// the table in every pass (any n).
template <bool kInRegs>
__device__ __forceinline__ bool low_end_select_impl(const uint32_t* keys, int n, int E, int* hist, uint32_t* bitmap,
                                                    uint32_t* cand_key, int* cand_idx, SelectSmem& sel, int* misc) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t* wmin = reinterpret_cast<uint32_t*>(sel.hist);          // (sel.hist is radix-select scratch)
    uint32_t* wmax = reinterpret_cast<uint32_t*>(sel.hist) + kFusedWarps;
    const int cnt = (n - tid + kFusedThreads - 1) / kFusedThreads;   // keys of this thread: tokens tid, tid + 512, ...
    constexpr int kSlots = kInRegs ? kFastKeys : 1;
    uint32_t kk[kSlots];
    if constexpr (kInRegs) {
#pragma unroll
        for (int j = 0; j < kFastKeys; ++j) kk[j] = j < cnt ? keys[tid + j * kFusedThreads] : 0xffffffffu;
    }
    {
        uint32_t lo = 0xffffffffu, hi = 0u;
        if constexpr (kInRegs) {
#pragma unroll
            for (int j = 0; j < kFastKeys; ++j) { lo = min(lo, kk[j]); if (j < cnt) hi = max(hi, kk[j]); }
        } else {
            for (int j = 0; j < cnt; ++j) { const uint32_t k = keys[tid + j * kFusedThreads]; lo = min(lo, k); hi = max(hi, k); }
        }
        // The E-th smallest key is at most the largest of any E distinct keys.  When at least E
        // threads hold keys, the thread minima are such keys, so the largest thread minimum bounds
        // it; otherwise the largest key does.  Keys above the bound share the top bin.
        const uint32_t cut = (n >= kFusedThreads && E <= kFusedThreads) ? lo : hi;
        const uint32_t wlo = __reduce_min_sync(0xffffffffu, lo);
        const uint32_t wcut = __reduce_max_sync(0xffffffffu, cnt > 0 ? cut : 0u);
        if (lane == 0) { wmin[warp] = wlo; wmax[warp] = wcut; }
    }
    __syncthreads();
    uint32_t kmin, kcut, shift;
    {
        const uint32_t lo = lane < kFusedWarps ? wmin[lane] : 0xffffffffu, hi = lane < kFusedWarps ? wmax[lane] : 0u;
        kmin = __reduce_min_sync(0xffffffffu, lo);
        kcut = __reduce_max_sync(0xffffffffu, hi);
        const int bits = 32 - __clz(kcut - kmin);   // significant bits of the range [kmin, kcut]
        shift = bits > 11 ? bits - 11 : 0;          // (key - kmin) >> shift < 2048 inside the range
    }
    // bin of a key: linear in the key over [kmin, kcut] (bins 0..2046), 2047 above; monotone
    auto bin_of = [kmin, kcut, shift](uint32_t k) { return k <= kcut ? min((k - kmin) >> shift, 2046u) : 2047u; };
    // (the top bin holds every key above the bound: the crossing is never there, so it is not counted)
    if constexpr (kInRegs) {
#pragma unroll
        for (int j = 0; j < kFastKeys; ++j) {
            const uint32_t b = bin_of(kk[j]);
            if (j < cnt && b != 2047u) atomicAdd(&hist[b], 1);
        }
    } else {
        for (int j = 0; j < cnt; ++j) {
            const uint32_t b = bin_of(keys[tid + j * kFusedThreads]);
            if (b != 2047u) atomicAdd(&hist[b], 1);
        }
    }
    __syncthreads();
    const int packed = find_crossing(hist, E, lane, warp, sel.warp_eq);
    const uint32_t bstar = static_cast<uint32_t>(packed >> 16);
    const int need = E - (packed & 0xffff);   // this many keys of the threshold bin go
    {
        int first = n;
        auto evict = [&](int i) { atomicOr(&bitmap[i >> 5], 1u << (i & 31)); first = min(first, i); };
        auto candidate = [&](uint32_t k, int i) {
            const int slot = atomicAdd(&misc[0], 1);
            if (slot < kFastCandCap) { cand_key[slot] = k; cand_idx[slot] = i; }
        };
        if constexpr (kInRegs) {
            unsigned m_below = 0, m_in = 0;           // bit j: this thread's j-th key is below / inside the bin
#pragma unroll
            for (int j = 0; j < kFastKeys; ++j) {
                const uint32_t b = bin_of(kk[j]);
                m_below |= (j < cnt && b < bstar) ? 1u << j : 0u;
                m_in |= (j < cnt && b == bstar) ? 1u << j : 0u;
            }
            if (packed >= 0 && (m_below | m_in)) {
                for (unsigned m = m_below; m; m &= m - 1) evict(tid + (__ffs(m) - 1) * kFusedThreads);
                for (unsigned m = m_in; m; m &= m - 1) {
                    const int i = tid + (__ffs(m) - 1) * kFusedThreads;
                    candidate(keys[i], i);
                }
            }
        } else if (packed >= 0) {
            for (int j = 0; j < cnt; ++j) {
                const int i = tid + j * kFusedThreads;
                const uint32_t k = keys[i], b = bin_of(k);
                if (b < bstar) evict(i);
                else if (b == bstar) candidate(k, i);
            }
        }
        first = __reduce_min_sync(0xffffffffu, first);   // one shared-memory atomic per warp, not per thread
        if (lane == 0 && first < n) atomicMin(&misc[1], first);
    }
    __syncthreads();
    const int ncand = misc[0];
    const bool ok = packed >= 0 && ncand <= kFastCandCap;   // the same in every thread
    if (ok) {
        int wfirst = n;
        for (int c = warp; c < ncand; c += kFusedWarps) {
            const uint32_t mk = cand_key[c];
            const int mi = cand_idx[c];
            int rank = 0;
            for (int q = lane; q < ncand; q += 32) {
                const uint32_t ok2 = cand_key[q];
                rank += (ok2 < mk) || (ok2 == mk && cand_idx[q] > mi);
            }
            rank = __reduce_add_sync(0xffffffffu, rank);
            if (lane == 0 && rank < need) { atomicOr(&bitmap[mi >> 5], 1u << (mi & 31)); wfirst = min(wfirst, mi); }
        }
        if (lane == 0 && wfirst < n) atomicMin(&misc[1], wfirst);
    }
    // Every thread has read misc[0] by now; whoever runs next (the full-table route resets misc) may write it.
    __syncthreads();
    return ok;
}
__device__ __noinline__ bool low_end_select_large(const uint32_t* keys, int n, int E, int* hist, uint32_t* bitmap,
                                                  uint32_t* cand_key, int* cand_idx, SelectSmem& sel, int* misc) {
    return low_end_select_impl<false>(keys, n, E, hist, bitmap, cand_key, cand_idx, sel, misc);   // (kept out of line: rare)
}
__device__ __forceinline__ bool low_end_select(const uint32_t* keys, int n, int E, int* hist, uint32_t* bitmap,
                                               uint32_t* cand_key, int* cand_idx, SelectSmem& sel, int* misc) {
    return n <= kFastKeys * kFusedThreads ? low_end_select_impl<true>(keys, n, E, hist, bitmap, cand_key, cand_idx, sel, misc)
                                          : low_end_select_large(keys, n, E, hist, bitmap, cand_key, cand_idx, sel, misc);
}

// Exact top-N over the whole key table by one CTA (every CTA of the cluster runs it on its own
// copy and gets the same answer): 2048-bin histogram, exact rank inside the threshold bin, radix
// select when that bin is crowded; then an ordered scan gives every kept row of this CTA's slice
// its destination (-1 = evicted) and misc[1] the index of the first evicted token.  With evict_bitmap the
// evicted tokens' bits are set there as well (cleared by the caller; pass seg_a = seg_b to skip the
// destinations).
__device__ __noinline__ void full_select_plan(const uint32_t* keys, int n, int N, int seg_a, int seg_b, int* hist,
                                              uint32_t* cand_key, int* cand_idx, int* dst_of, SelectSmem& sel, int* misc,
                                              uint32_t* evict_bitmap = nullptr) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int b = tid; b < kBins; b += kFusedThreads) hist[b] = 0;
    if (tid == 0) { misc[0] = 0; misc[1] = n; }
    __syncthreads();
    // thread t owns the tokens [i0, i1): an odd stride keeps the shared-memory reads conflict-free
    const int per = ((n + kFusedThreads - 1) / kFusedThreads) | 1;
    const int i0 = min(n, tid * per), i1 = min(n, i0 + per);
    for (int i = i0; i < i1; ++i) atomicAdd(&hist[key_bin(keys[i])], 1);
    __syncthreads();
    {
        // thread t owns bins 2047-4t .. 2044-4t (descending); find the bin holding rank N
        int c4[4], tot = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) { c4[q] = hist[kBins - 1 - 4 * tid - q]; tot += c4[q]; }
        int incl = tot;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) sel.warp_gt[warp] = incl;
        __syncthreads();
        int before = 0;
        for (int w = 0; w < warp; ++w) before += sel.warp_gt[w];
        incl += before;
        const int excl = incl - tot;
        if (excl < N && N <= incl) {
            int above = excl;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (above < N && N <= above + c4[q]) { sel.bcast[0] = kBins - 1 - 4 * tid - q; sel.bcast[1] = above; }
                above += c4[q];
            }
        }
        __syncthreads();
    }
    const int bstar = sel.bcast[0];
    const int need = N - sel.bcast[1];       // tokens of the threshold bin that are kept, >= 1
    for (int j = 0; j < per; ++j) {          // same trip count in every lane: the ballot is warp-wide
        const int i = i0 + j;
        const uint32_t k = i < i1 ? keys[i] : 0u;
        const bool inbin = i < i1 && key_bin(k) == bstar;
        const unsigned peers = __ballot_sync(0xffffffffu, inbin);
        if (peers != 0) {                    // one shared-memory atomic per warp, not per candidate
            const int leader = __ffs(peers) - 1;
            int base = 0;
            if (lane == leader) base = atomicAdd(&misc[0], __popc(peers));
            base = __shfl_sync(0xffffffffu, base, leader);
            const int slot = base + __popc(peers & ((1u << lane) - 1u));
            if (inbin && slot < kCandCap) { cand_key[slot] = k; cand_idx[slot] = i; }
        }
    }
    __syncthreads();
    Threshold th;
    const int ncand = misc[0];
    if (ncand <= kCandCap) {
        // exact rank among the candidates under (key desc, index asc): one candidate per warp at a
        // time, its comparisons spread over the lanes
        for (int c = warp; c < ncand; c += kFusedWarps) {
            const uint32_t mk = cand_key[c];
            const int mi = cand_idx[c];
            int rank = 0, eq_older = 0;
            for (int q = lane; q < ncand; q += 32) {
                const uint32_t ok = cand_key[q];
                const int oi = cand_idx[q];
                rank += (ok > mk) || (ok == mk && oi < mi);
                eq_older += (ok == mk && oi <= mi);
            }
            rank = __reduce_add_sync(0xffffffffu, rank);
            eq_older = __reduce_add_sync(0xffffffffu, eq_older);
            if (lane == 0 && rank == need - 1) { misc[3] = static_cast<int>(mk); misc[2] = eq_older; }
        }
        __syncthreads();
        th.key = static_cast<uint32_t>(misc[3]);
        th.need_eq = misc[2];
    } else {
        th = block_radix_select<kFusedThreads>(keys, n, N, sel);
    }
    int gt = 0, eq = 0;
    for (int i = i0; i < i1; ++i) { const uint32_t k = keys[i]; gt += k > th.key; eq += k == th.key; }
    int pre_gt, pre_eq, tot_gt, tot_eq;
    block_exclusive_scan2<kFusedThreads>(gt, eq, sel, pre_gt, pre_eq, tot_gt, tot_eq);   // syncs: hist is dead
    int local_first = n;
    for (int i = i0; i < i1; ++i) {
        const uint32_t k = keys[i];
        const bool is_eq = k == th.key;
        const bool keep = k > th.key || (is_eq && pre_eq < th.need_eq);
        if (i >= seg_a && i < seg_b) dst_of[i - seg_a] = keep ? pre_gt + min(pre_eq, th.need_eq) : -1;
        if (!keep && evict_bitmap) atomicOr(&evict_bitmap[i >> 5], 1u << (i & 31));
        if (!keep) local_first = min(local_first, i);
        pre_gt += k > th.key;
        pre_eq += is_eq;
    }
    if (local_first < n) atomicMin(&misc[1], local_first);
    __syncthreads();
}

// The anchor's running sum (App. B.1, first expression, carried across steps) is kept so that it cannot drift:
// EVERY ROW'S TERM IS A FIXED BIT PATTERN -- the fp32 products of the row's bf16 elements and the row's fp32
// reciprocal norm, both functions of the row alone -- and terms are added and subtracted in double precision.  A
// row that enters the cache adds exactly what it takes away when it is evicted, and no fp32 partial sum of the
// size of the anchor appears anywhere (an anchor over keys that point in many directions is a cancelling sum;
// fp32 partial sums would limit it, and with it every score, to about 1e-7 / ||mu||).
// warp_row_terms (below) forms these terms; both fused kernels and the staged kernels use the same products.

// Evicted tokens before each word of the bitmap: wlocal[w] = number of set bits in words [0, w).  All threads
// call; uses sel.warp_gt, sel.hist[32..48) and misc[5], misc[6]; ends with a CTA barrier.
__device__ __forceinline__ void bitmap_prefix(const uint32_t* bitmap, int nwords, int* wlocal, SelectSmem& sel, int* misc) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int* wbase = sel.hist + 2 * kFusedWarps;
    if (nwords <= kFusedThreads) {   // one word per thread: every warp scans the 16 warp totals itself
        const int pc = tid < nwords ? __popc(bitmap[tid]) : 0;
        int incl = pc;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) sel.warp_gt[warp] = incl;
        __syncthreads();
        const int t2 = lane < kFusedWarps ? sel.warp_gt[lane] : 0;
        int incl2 = t2;
#pragma unroll
        for (int o = 1; o < 16; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, incl2, o); if (lane >= o) incl2 += v; }
        const int base = __shfl_sync(0xffffffffu, incl2 - t2, warp);   // evicted tokens before this warp's 32 words
        if (tid < nwords) wlocal[tid] = base + incl - pc;
        __syncthreads();
        return;
    }
    for (int w0 = 0; w0 < nwords; w0 += kFusedThreads) {
        const int wi = w0 + tid;
        const int pc = wi < nwords ? __popc(bitmap[wi]) : 0;
        int incl = pc;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) sel.warp_gt[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            const int t2 = lane < kFusedWarps ? sel.warp_gt[lane] : 0;
            int incl2 = t2;
#pragma unroll
            for (int o = 1; o < 16; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, incl2, o); if (lane >= o) incl2 += v; }
            if (lane < kFusedWarps) wbase[lane] = incl2 - t2 + (w0 > 0 ? misc[5] : 0);
            if (lane == kFusedWarps - 1) misc[6] = incl2 + (w0 > 0 ? misc[5] : 0);
        }
        __syncthreads();
        if (wi < nwords) wlocal[wi] = wbase[warp] + incl - pc;   // evicted tokens before word wi
        if (tid == 0) misc[5] = misc[6];
        __syncthreads();
    }
}

// ||mu|| from the fp32 anchor in shared memory, computed by every warp in the same order.
__device__ __forceinline__ float anchor_norm(const float* mu, int lane) {
    const float4 c4 = reinterpret_cast<const float4*>(mu)[lane];
    float v = fmaf(c4.w, c4.w, fmaf(c4.z, c4.z, fmaf(c4.y, c4.y, c4.x * c4.x)));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return sqrtf(v);
}
// Steps a1 + a2 for one landed tile when the anchor is known beforehand: norm and dot product of its 16 rows in
// one pass, four rows per row group; the keys go to keys_seg[local row].  The whole warp calls.
__device__ __forceinline__ void score_tile(const uint4* rows, int tile, int rs, int t, int sub, const float2 (&w)[8], float m,
                                           float eps, uint32_t* keys_seg) {
    float vs[4];   // this lane's shares of the tile's four rows of its row group
    double vd[4];
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int lr = tile * kTileRows + it * 4 + sub;
        uint4 a = make_uint4(0, 0, 0, 0), b = a;
        if (lr < rs) { a = rows[lr * kRowVec + t]; b = rows[lr * kRowVec + t + 8]; }
        lane_sumsq_dot(a, b, w, vs[it], vd[it]);
    }
    const uint32_t key = score4(vs, vd, t, m, eps);
    const int lr = tile * kTileRows + (t >> 1) * 4 + sub;
    if (!(t & 1) && lr < rs) keys_seg[lr] = key;   // (both lanes of a pair hold the row's key)
}

// The canonical form of a row's anchor terms inside the fused kernel: ONE WARP PER ROW, lane l holding channels
// 4l .. 4l+3 (two packed words).  ||k||^2 = the lanes' four-term chains added by the xor butterfly 16, 8, 4, 2, 1;
// 1/||k|| by the approximate reciprocal square root (or min with 1/eps); the four terms are the fp32 products,
// added to acc in double.  Every place that adds or removes a row's terms uses this function, so that a row takes
// away exactly what it brought.  The whole warp calls; `active` is warp-uniform.
__device__ __forceinline__ void warp_row_terms(uint2 wds, bool active, float inv_eps, bool raw, double (&acc)[4]) {
    const float x0 = bf16_lo(wds.x), x1 = bf16_hi(wds.x), x2 = bf16_lo(wds.y), x3 = bf16_hi(wds.y);
    float ss = fmaf(x3, x3, fmaf(x2, x2, fmaf(x1, x1, x0 * x0)));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (active) {
        const float inv = raw ? 1.0f : fminf(approx_rsqrt(ss), inv_eps);
        acc[0] += static_cast<double>(__fmul_rn(x0, inv)); acc[1] += static_cast<double>(__fmul_rn(x1, inv));
        acc[2] += static_cast<double>(__fmul_rn(x2, inv)); acc[3] += static_cast<double>(__fmul_rn(x3, inv));
    }
}
// The 16 warps' four sums per lane (channels 4l .. 4l+3) added up over the CTA in a fixed order through an
// [8][128] table of doubles: warps 0..7 store their sums, warps 8..15 add theirs to the row of warp w - 8, and
// channel c's total is the sum of the eight rows in order.  Returns the total in threads tid < 128 (0 elsewhere).
// Two CTA barriers inside; the caller synchronises before the table is reused.
__device__ __forceinline__ double cta_sum_of_warp_sums(const double (&acc)[4], double* table, int tid) {
    const int warp = tid >> 5, lane = tid & 31;
    double2* row = reinterpret_cast<double2*>(table + (warp & 7) * kHeadDim + 4 * lane);
    if (warp < 8) { row[0] = make_double2(acc[0], acc[1]); row[1] = make_double2(acc[2], acc[3]); }
    __syncthreads();
    if (warp >= 8) {
        const double2 a = row[0], b = row[1];
        row[0] = make_double2(a.x + acc[0], a.y + acc[1]); row[1] = make_double2(b.x + acc[2], b.y + acc[3]);
    }
    __syncthreads();
    double s = 0.0;
    if (tid < kHeadDim) {
#pragma unroll
        for (int w = 0; w < 8; ++w) s += table[w * kHeadDim + tid];
    }
    return s;
}

// kRegRows = rows per row group that live in registers (the host picks the smallest instance that
// holds a slice together with the shared-memory rows).
//
// kOnePass: the anchor is known before the keys are scored.  The library keeps, per unit, the sum of the terms
// k/||k|| over the rows in the cache (App. B.1, expr. 1, split over time): a step's sum over its n rows is that
// running sum plus the sum over the B block rows, so only the block has to be normalised before scoring, norm
// and dot product of a row are taken in one pass, and the first cluster barrier, the anchor exchange and the
// second pass over the rows disappear.  The anchor of the cluster's NEXT unit is formed while this unit's V rows
// are on their way in, and the next unit's K tiles are scored by the warp that owns them as soon as they have
// landed behind the V rows going out: the scoring runs under the copies instead of after them.  Every step
// (either kind) subtracts the evicted rows' terms again: each CTA leaves the change it saw in anchor_delta, and
// the next step folds the deltas into the running sum, in double precision and in a fixed order.
// kOnePass = false recomputes the anchor from all n rows (first evicting step, after set_len / reset / appends,
// and periodically).
//
// kPreRows: block rows per warp and kind that are requested before the K stores and held in registers across them
// (the rest is read after the stores, latency exposed).  The host picks 1 when a CTA's share of the block is at
// most one row per warp (B <= 16 C) -- the registers this frees shorten the store loop -- and 4 otherwise.
template <int kRegRows, bool kOnePass, int kPreRows>
__global__ void __launch_bounds__(kFusedThreads, 1) fused_evict_kernel(const FusedParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int C = p.cluster;
    const FusedLayout L = fused_layout(p.smem_rows, p.nkeys, C);
    uint4* rows = reinterpret_cast<uint4*>(smem + L.rows);
    uint32_t* keys = reinterpret_cast<uint32_t*>(smem + L.keys);
    int* hist = reinterpret_cast<int*>(smem + L.work);
    int* dst_of = reinterpret_cast<int*>(smem + L.work);
    double* partials = reinterpret_cast<double*>(smem + L.xchg + 2 * kCandCap * 4);   // [C][128], filled by the peers: the anchor
                                                                                    // partials of a two-pass step, the shares of the
                                                                                    // next unit's block sum in a one-pass step
    uint32_t* cand_key = reinterpret_cast<uint32_t*>(smem + L.xchg);
    int* cand_idx = reinterpret_cast<int*>(smem + L.xchg) + kCandCap;
    SelectSmem& sel = *reinterpret_cast<SelectSmem*>(smem + L.sel);
    float* mu_buf = reinterpret_cast<float*>(smem + L.mu);   // two anchors: this unit's and the next unit's
    int* misc = reinterpret_cast<int*>(smem + L.misc);   // 0 ncand, 1 first_evicted, 2 need_eq, 3 threshold key, 5/6 prefix carry
    const uint32_t rows_sa = smem_addr(rows), mbar_sa = smem_addr(smem + L.mbar);
    const uint32_t keys_sa = smem_addr(keys), partials_sa = smem_addr(partials);
    // scratch that the dead key table lends between the selection and the third cluster barrier (no peer writes the
    // table in that window): every warp's sums of the terms that left and of the next block's terms
    double* gone_tab = reinterpret_cast<double*>(keys);                 // [8][128]: warps w and w + 8 share row w
    double* next_tab = gone_tab + (kFusedWarps / 2) * kHeadDim;         // [8][128]
    uint4* warp_row = reinterpret_cast<uint4*>(smem + L.xchg);          // [16 warps][16 words]: a register-resident row, re-read
                                                                        // one warp per row (the candidates' area, dead by then)

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = tid >> 3, t = tid & 7, sub = lane >> 3;
    const int crank = static_cast<int>(cluster_ctarank());
    const int cluster_id = blockIdx.x / C, nclusters = gridDim.x / C;
    const int len = p.len, B = p.B, N = p.N, n = len + B, E = n - N;   // E tokens are evicted
    const float inv_eps = 1.0f / p.eps;
    const bool raw = p.raw_anchor != 0;
    const int nwords = (n + 31) >> 5;
    uint32_t* bitmap = reinterpret_cast<uint32_t*>(smem + L.bitmap);
    int* wlocal = reinterpret_cast<int*>(smem + L.bitmap) + ((p.nkeys + 31) >> 5);
    Slice sl;
    sl.seg_a = min(n, crank * p.rows_per_cta);
    sl.seg = min(n, sl.seg_a + p.rows_per_cta) - sl.seg_a;
    sl.rs = min(sl.seg, p.smem_rows);
    sl.ntiles = (sl.rs + kTileRows - 1) / kTileRows;
    const int seg_a = sl.seg_a, seg = sl.seg, rs = sl.rs, ntiles = sl.ntiles;
    // Shared-memory rows are handled tile by tile (16 rows); warp w owns tiles w, w+16, w+32, ... in
    // every phase, so a tile is loaded, read, written out and refilled by one warp: the hand-over of
    // a tile from its readers to the copy engine needs a __syncwarp, never a CTA-wide barrier.

    if (tid == 0) {
        for (int j = 0; j <= kMaxTiles; ++j) mbar_init(mbar_sa + 8 * j, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    uint32_t parity = 0;   // bit s: phase parity the next wait on this warp's s-th tile expects
    uint32_t xparity = 0;  // phase parity of the key exchange's barrier

    // All clusters start together and do identical work per unit, so left alone they stay in lock
    // step: every SM loads at the same moment, then every SM computes while HBM idles.  Starting
    // cluster c a fraction of a unit's duration late spreads the memory phases over time.  Clusters
    // with the lower ids are also the ones that may own one unit more, so the delay mostly fills
    // slack that the uneven unit count leaves anyway.  The wait is bounded.
    if (p.stagger_ns != 0 && cluster_id != 0) {
        const unsigned long long t0 = global_timer_ns();
        const unsigned long long wait_ns = static_cast<unsigned long long>(p.stagger_ns) * static_cast<unsigned>(cluster_id);
        for (int spin = 0; spin < (1 << 16) && global_timer_ns() - t0 < wait_ns; ++spin) __nanosleep(100);
    }

    KD_STAMP_DECL
    constexpr int kRegSlots = kRegRows > 0 ? kRegRows : 1;   // no zero-sized arrays in device code
    uint4 ra[kRegSlots], rb[kRegSlots];   // register-resident rows: local row rs + 64k + g
    // K of the cluster's first unit: tiles by the copy engine, the rest by plain loads
    if (cluster_id < p.U) {
        if (lane < kTilesPerWarp && warp + kFusedWarps * lane < ntiles)
            issue_tile(p.k_cache, p.new_k, cluster_id, len, B, N, sl, warp + kFusedWarps * lane, rows_sa, mbar_sa);
#pragma unroll
        for (int k = 0; k < kRegRows; ++k) {
            const int lr = rs + k * kGroups + g;
            ra[k] = make_uint4(0, 0, 0, 0); rb[k] = ra[k];
            if (lr < seg) {
                const uint4* row = concat_row(p.k_cache, p.new_k, cluster_id, seg_a + lr, len, B, N);
                ra[k] = row[t]; rb[k] = row[t + 8];
            }
        }
    }

    // One-pass steps.  The B block rows of a unit are normalised once per cluster: CTA r takes block rows
    // [b_lo, b_hi), pushes its share of their sum of terms into every peer's table (DSMEM), and after a cluster
    // barrier every CTA adds the C shares in rank order to the folded running sum: the same anchor bits everywhere.
    const int b_per = (B + C - 1) / C;
    const int b_lo = min(B, crank * b_per), b_hi = min(B, b_lo + b_per);
    // (this CTA's own share of a unit's block sum is not kept in a register: every CTA pushes its share to all CTAs
    // of the cluster, itself included, so it stays readable in row `crank` of this CTA's own table until the next push)
    bool tiles_scored = false;   // this unit's tiles were scored behind the previous unit's V rows
    int cur = 0;                 // which of the two anchor buffers holds this unit's anchor
    auto fold_running_sum = [&](int uu) -> double {   // threads tid < 128
        double a = p.anchor_in[static_cast<size_t>(uu) * kHeadDim + tid];
        double dl[kMaxCluster];
#pragma unroll
        for (int c = 0; c < kMaxCluster; ++c)
            dl[c] = c < C ? p.anchor_delta[(static_cast<size_t>(uu) * C + c) * kHeadDim + tid] : 0.0;
#pragma unroll
        for (int c = 0; c < kMaxCluster; ++c) a += dl[c];   // rank order; absent ranks add 0
        if (crank == 0) p.anchor_out[static_cast<size_t>(uu) * kHeadDim + tid] = a;   // the cached rows' sum, folded
        return a;
    };
    auto push_share = [&](double v) {   // threads tid < 128: this CTA's row of every peer's table
        const uint32_t slot = partials_sa + 8 * (crank * kHeadDim + tid);
        for (int c = 0; c < C; ++c) st_cluster_f64(map_to_cta(slot, c), v);
    };
    auto anchor_from_shares = [&](double a, float* mu_out) {   // threads tid < 128, after the cluster barrier
        double bs = 0.0;
        for (int c = 0; c < C; ++c) bs += partials[c * kHeadDim + tid];
        mu_out[tid] = static_cast<float>((a + bs) / static_cast<double>(n));
    };
    if (kOnePass && cluster_id < p.U) {   // the first unit's anchor (the work area is free before the first unit)
        double folded = 0.0;
        if (tid < kHeadDim) folded = fold_running_sum(cluster_id);
        {
            double acc[4] = {0.0, 0.0, 0.0, 0.0};
            const uint4* blk = p.new_k + static_cast<size_t>(cluster_id) * B * kRowVec;
            for (int j = b_lo + warp; j < b_hi; j += kFusedWarps)   // (warp-uniform)
                warp_row_terms(reinterpret_cast<const uint2*>(blk + static_cast<size_t>(j) * kRowVec)[lane], true, inv_eps, raw, acc);
            const double first_share = cta_sum_of_warp_sums(acc, gone_tab, tid);   // (nobody uses the key table before the first unit's scores)
            __syncthreads();   // the table is free again before any key is written
            if (tid < kHeadDim) push_share(first_share);
        }
        cluster_sync_all();
        if (tid < kHeadDim) anchor_from_shares(folded, mu_buf);
        __syncthreads();
    }

    // one-pass scoring of the register-resident rows (they hold the K rows of the unit to be scored), four at a time
    auto score_reg_rows = [&](const float2 (&w)[8], float m) {
#pragma unroll
        for (int k0 = 0; k0 < kRegRows; k0 += 4) {
            float vs[4];
            double vd[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (k0 + i < kRegRows) lane_sumsq_dot(ra[k0 + i], rb[k0 + i], w, vs[i], vd[i]);
                else { vs[i] = 0.f; vd[i] = 0.0; }
            }
            const uint32_t key = score4(vs, vd, t, m, p.eps);
            const int lr = rs + (k0 + (t >> 1)) * kGroups + g;
            if (!(t & 1) && k0 + (t >> 1) < kRegRows && lr < seg) keys[seg_a + lr] = key;
        }
    };
    KD_STAMP(0);
    for (int u = cluster_id; u < p.U; u += nclusters) {
        const int un = u + nclusters;   // the unit this cluster serves next
        float* mu_sh = mu_buf + cur * kHeadDim;
        if constexpr (kOnePass) {
            // ------------------------------------------------------------ a1 + a2 in one pass: keys of this slice
            // (every unit but the cluster's first was scored behind the previous unit's V rows)
            if (!tiles_scored) {
                float2 w[8];
                load_anchor(mu_sh, t, w);
                const float m = anchor_norm(mu_sh, lane);
#pragma unroll 1
                for (int s = 0; s < kTilesPerWarp; ++s) {
                    const int tile = warp + kFusedWarps * s;
                    if (tile >= ntiles) break;
                    mbar_wait(mbar_sa + 8 * tile, (parity >> s) & 1u, p.status);
                    parity ^= 1u << s;
                    score_tile(rows, tile, rs, t, sub, w, m, p.eps, keys + seg_a);
                }
                score_reg_rows(w, m);
            }
        } else {
            // ------------------------------------------------------------ a1: norms and anchor partial
            float rn[kRegSlots];
            double wide[16];   // this thread's sums, carried in double above the four rows of a tile
#pragma unroll
            for (int j = 0; j < 16; ++j) wide[j] = 0.0;
#pragma unroll 1
            for (int s = 0; s < kTilesPerWarp; ++s) {
                const int tile = warp + kFusedWarps * s;
                if (tile >= ntiles) break;
                mbar_wait(mbar_sa + 8 * tile, (parity >> s) & 1u, p.status);
                parity ^= 1u << s;
                float2 acc[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) acc[q] = make_float2(0.f, 0.f);
#pragma unroll 1
                for (int half = 0; half < 2; ++half) {
                    uint4 a[2], b[2];
#pragma unroll
                    for (int it = 0; it < 2; ++it) {
                        const int lr = tile * kTileRows + (2 * half + it) * 4 + sub;
                        a[it] = make_uint4(0, 0, 0, 0); b[it] = a[it];
                        if (lr < rs) { a[it] = rows[lr * kRowVec + t]; b[it] = rows[lr * kRowVec + t + 8]; }
                    }
#pragma unroll
                    for (int it = 0; it < 2; ++it) {
                        const int lr = tile * kTileRows + (2 * half + it) * 4 + sub;
                        const float r = row_a1(a[it], b[it], lr < rs, inv_eps, acc, raw);
                        if (lr < rs && t == 0) keys[seg_a + lr] = __float_as_uint(r);   // parked in the row's key slot until a2
                    }
                }
#pragma unroll
                for (int q = 0; q < 8; ++q) { wide[2 * q] += static_cast<double>(acc[q].x); wide[2 * q + 1] += static_cast<double>(acc[q].y); }
            }
            {
                float2 acc[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) acc[q] = make_float2(0.f, 0.f);
#pragma unroll
                for (int k = 0; k < kRegRows; ++k) rn[k] = row_a1(ra[k], rb[k], rs + k * kGroups + g < seg, inv_eps, acc, raw);
#pragma unroll
                for (int q = 0; q < 8; ++q) { wide[2 * q] += static_cast<double>(acc[q].x); wide[2 * q + 1] += static_cast<double>(acc[q].y); }
            }
            // CTA reduction in double (the key table holds the parked norms, so the 8 KB work area serves, in two rounds)
            {
                const double s = cta_channel_sum<1>(wide, reinterpret_cast<double*>(smem + L.work), tid);
                if (tid < kHeadDim) {
                    const uint32_t slot = partials_sa + 8 * (crank * kHeadDim + tid);
                    for (int c = 0; c < C; ++c) st_cluster_f64(map_to_cta(slot, c), s);   // this CTA's row of every peer's table
                }
            }
            cluster_sync_all();   // (1) all partials delivered; every K row of the unit is on chip
            if (tid < kHeadDim) {
                double s = 0.0;
                for (int c = 0; c < C; ++c) s += partials[c * kHeadDim + tid];   // rank order: same bits in every CTA
                mu_sh[tid] = static_cast<float>(s / static_cast<double>(n));
                if (crank == 0) p.anchor_out[static_cast<size_t>(u) * kHeadDim + tid] = s;   // sum over all n rows
            }
            __syncthreads();
            // ------------------------------------------------------------ a2: keys of this slice into the table
            float2 w[8];
            load_anchor(mu_sh, t, w);
            const float m = anchor_norm(mu_sh, lane);
#pragma unroll 1
            for (int s = 0; s < kTilesPerWarp; ++s) {
                const int tile = warp + kFusedWarps * s;
                if (tile >= ntiles) break;
#pragma unroll 1
                for (int half = 0; half < 2; ++half) {
                    uint4 a[2], b[2];
                    float r[2];
#pragma unroll
                    for (int it = 0; it < 2; ++it) {
                        const int lr = tile * kTileRows + (2 * half + it) * 4 + sub;
                        a[it] = make_uint4(0, 0, 0, 0); b[it] = a[it]; r[it] = 0.f;
                        if (lr < rs) { a[it] = rows[lr * kRowVec + t]; b[it] = rows[lr * kRowVec + t + 8]; r[it] = __uint_as_float(keys[seg_a + lr]); }
                    }
#pragma unroll
                    for (int it = 0; it < 2; ++it) {
                        const int lr = tile * kTileRows + (2 * half + it) * 4 + sub;
                        const uint32_t key = row_a2(a[it], b[it], w, m, r[it], p.eps);
                        if (lr < rs && t == 0) keys[seg_a + lr] = key;
                    }
                }
            }
#pragma unroll
            for (int k = 0; k < kRegRows; ++k) {
                const uint32_t key = row_a2(ra[k], rb[k], w, m, rn[k], p.eps);
                const int lr = rs + k * kGroups + g;
                if (lr < seg && t == 0) keys[seg_a + lr] = key;
            }
        }   // kOnePass
        KD_STAMP(1);
        // this slice's keys -> every peer's table: one bulk copy per peer, counted on the PEER's exchange barrier; a CTA
        // goes on as soon as its own table is complete (n - seg keys have landed), no cluster-wide barrier.  The
        // peers' tables are free: nobody writes a unit's keys before it has passed the previous unit's third barrier.
        fence_proxy_async_smem();   // this thread's keys, in front of the copy engine's reads
        __syncthreads();
        if (tid == 0) {
            // (a bulk copy moves multiples of 16 bytes: a ragged last slice is sent with up to three entries of
            // padding, which land beyond key n - 1 inside the sender's own part of the table and are never read)
            const uint32_t xbar = mbar_sa + 8 * kMaxTiles;
            uint32_t expected = 0;
            for (int c = 0; c < C; ++c) {
                const int a = min(n, c * p.rows_per_cta), sg = min(n, a + p.rows_per_cta) - a;
                if (c != crank) expected += static_cast<uint32_t>((sg + 3) & ~3) * 4u;
            }
            mbar_expect_tx(xbar, expected);   // what the peers will send here
            if (seg > 0) {
                const uint32_t bytes = static_cast<uint32_t>((seg + 3) & ~3) * 4u;
                for (int c = 1; c < C; ++c) {
                    const uint32_t peer = static_cast<uint32_t>(crank + c < C ? crank + c : crank + c - C);
                    bulk_push(map_to_cta(keys_sa + 4 * seg_a, peer), keys_sa + 4 * seg_a, bytes, map_to_cta(xbar, peer));
                }
            }
        }
        {
            float* sc = p.scores + static_cast<size_t>(u) * p.nmax + seg_a;   // fp32 scores to global scratch, coalesced
            for (int lr = tid; lr < seg; lr += kFusedThreads) __stcs(&sc[lr], key_score(keys[seg_a + lr]));
            for (int b = tid; b < kBins; b += kFusedThreads) hist[b] = 0;
            for (int wd = tid; wd < nwords; wd += kFusedThreads) bitmap[wd] = 0;
            if (tid == 0) { misc[0] = 0; misc[1] = n; }
        }
        mbar_wait(mbar_sa + 8 * kMaxTiles, xparity, p.status);   // (2) this CTA's key table holds all n keys
        xparity ^= 1u;
        __syncthreads();   // (the zeroing above is complete as well)
        KD_STAMP(2);
        if (p.window > 0) {
            // sliding window (Sec. 3.2): the last `window` tokens get the largest possible key, so they are
            // never among the E smallest; the scores in global scratch stay what they are
            __syncthreads();   // this CTA's score write-out has read its keys
            for (int i = n - p.window + tid; i < n; i += kFusedThreads) keys[i] = 0xffffffffu;
            __syncthreads();
        }
        // ------------------------------------------------------------ a3 + plan: who is evicted, where every kept row goes
        {
            // the evicted tokens' bits: selection at the low end of the table, or (crowded threshold bin, large
            // unit) the full-table route; then prefix counts over the bitmap give every kept row of the slice
            // its destination
            const bool planned = low_end_select(keys, n, E, hist, bitmap, cand_key, cand_idx, sel, misc);
            if (!planned) {
                for (int wd = tid; wd < nwords; wd += kFusedThreads) bitmap[wd] = 0;   // (the attempt may have marked some)
                __syncthreads();
                full_select_plan(keys, n, N, 0, 0, hist, cand_key, cand_idx, nullptr, sel, misc, bitmap);
            }
            bitmap_prefix(bitmap, nwords, wlocal, sel, misc);
            for (int lr = tid; lr < seg; lr += kFusedThreads) {
                const int i = seg_a + lr, w = i >> 5;
                const uint32_t wd = bitmap[w], bit = 1u << (i & 31);
                dst_of[lr] = (wd & bit) ? -1 : i - (wlocal[w] + __popc(wd & (bit - 1)));
            }
            __syncthreads();
        }
        KD_STAMP(3);
        const int first_evicted = misc[1];
        const int first_moved = min(first_evicted, len);   // block rows always move into the cache
        const int skip_local = first_moved - seg_a;        // local rows below this keep their place
        if (crank == 0 && tid == 0) {
            p.first_evicted[u] = first_evicted;
            atomicAdd(p.moved_rows, static_cast<unsigned long long>(N - first_moved));
        }
        for (int lr = tid; lr < seg; lr += kFusedThreads) {   // kept-index list, coalesced (destinations ascend with lr)
            const int d = dst_of[lr];
            if (d >= 0) {
                __stcs(&p.kept_idx[static_cast<size_t>(u) * N + d], seg_a + lr);
                if (p.kept_mirror) p.kept_mirror[static_cast<size_t>(u) * N + d] = seg_a + lr;
            }
        }
        KD_STAMP(4);
        // ------------------------------------------------------------ a4: K rows out, V rows in behind them; the rows that leave
        // the cache and this CTA's range of the next block turn into anchor terms along the way
        // This CTA's delta to the running sum: its share of the block that came in (one-pass steps) minus the terms
        // of (a) the evicted cache rows of its slice -- each taken by the warp that holds it, from the tile or the
        // registers, just before the K stores hand the tile on -- and (b) the evicted block rows of its range of the
        // block, which stay readable in global memory (warp w takes rows w, w + 16, ... of the range).
        double acc_g[4] = {0.0, 0.0, 0.0, 0.0}, acc_n[4] = {0.0, 0.0, 0.0, 0.0};
        const bool next_share = kOnePass && un < p.U;
        const uint4* blk_u = p.new_k + static_cast<size_t>(u) * B * kRowVec;
        const uint4* blk_n = p.new_k + static_cast<size_t>(next_share ? un : u) * B * kRowVec;
        auto block_row_evicted = [&](int j) { const int i = len + j; return j < b_hi && ((bitmap[i >> 5] >> (i & 31)) & 1u) != 0; };
        uint2 pre_e[kPreRows], pre_n[kPreRows];   // requested now, used after the K stores
#pragma unroll
        for (int k = 0; k < kPreRows; ++k) {
            const int j = b_lo + warp + k * kFusedWarps;
            pre_e[k] = make_uint2(0, 0); pre_n[k] = pre_e[k];
            if (block_row_evicted(j)) pre_e[k] = reinterpret_cast<const uint2*>(blk_u + static_cast<size_t>(j) * kRowVec)[lane];
            if (next_share && j < b_hi) pre_n[k] = reinterpret_cast<const uint2*>(blk_n + static_cast<size_t>(j) * kRowVec)[lane];
        }
        double folded_next = 0.0;
        if (next_share && tid < kHeadDim) folded_next = fold_running_sum(un);   // (its loads arrive under the stores)
        {
            // (row stores are streaming stores: a written row is not touched again in this step; measured 0.5 % on the step)
            uint4* out = p.k_cache + static_cast<size_t>(u) * N * kRowVec;
            if (kOnePass && crank == 0 && un + nclusters < p.U) {   // the block rows of the unit after next towards L2
                const char* nb = reinterpret_cast<const char*>(p.new_k + static_cast<size_t>(un + nclusters) * B * kRowVec);
                for (int o = tid * 128; o < B * kRowBytes; o += kFusedThreads * 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(nb + o));
            }
#pragma unroll
            for (int k = 0; k < kRegRows; ++k) {
                const int lr = rs + k * kGroups + g;
                const bool vis = lr < seg && lr >= skip_local;
                const int d = vis ? dst_of[lr] : -1;
                if (d >= 0 && KD_ROW_OK(d, N, p.status)) { __stcs(&out[d * kRowVec + t], ra[k]); __stcs(&out[d * kRowVec + t + 8], rb[k]); }
                // evicted cache rows among the warp's four (a nibble of the bitmap says whether there is any): one at a
                // time through the warp's scratch row, re-read one warp per row
                const int i4 = seg_a + rs + k * kGroups + 4 * warp;   // the warp's four rows are tokens i4 .. i4 + 3 (i4 % 4 == 0)
                const bool any_gone = i4 < len && ((bitmap[i4 >> 5] >> (i4 & 31)) & 0xfu) != 0;   // (warp-uniform)
                for (unsigned gm = any_gone ? __ballot_sync(0xffffffffu, vis && d < 0 && seg_a + lr < len) & 0x01010101u : 0u; gm; gm &= gm - 1) {
                    const int gsub = (__ffs(gm) - 1) >> 3;
                    __syncwarp();
                    if (sub == gsub) { warp_row[warp * kRowVec + t] = ra[k]; warp_row[warp * kRowVec + t + 8] = rb[k]; }
                    __syncwarp();
                    warp_row_terms(reinterpret_cast<const uint2*>(warp_row + warp * kRowVec)[lane], true, inv_eps, raw, acc_g);
                }
                if (vis) {
                    const uint4* row = concat_row(p.v_cache, p.new_v, u, seg_a + lr, len, B, N);
                    ra[k] = row[t]; rb[k] = row[t + 8];
                }
            }
#pragma unroll 1
            for (int s = 0; s < kTilesPerWarp; ++s) {
                const int tile = warp + kFusedWarps * s;
                if (tile >= ntiles) break;
                if (min(rs, (tile + 1) * kTileRows) <= skip_local) continue;   // no row of the tile moves
                // the bitmap bits of the tile's 16 tokens (they may straddle two words; a word past the end only adds
                // bits that the exact test below rejects)
                const int i16 = seg_a + tile * kTileRows;
                const unsigned gone16 = i16 < len ? __funnelshift_r(bitmap[i16 >> 5], bitmap[(i16 >> 5) + 1], i16 & 31) & 0xffffu : 0u;   // (warp-uniform)
#pragma unroll
                for (int it = 0; it < 4; ++it) {
                    const int lr = tile * kTileRows + it * 4 + sub;
                    const bool vis = lr < rs && lr >= skip_local;
                    const int d = vis ? dst_of[lr] : -1;
                    if (d >= 0 && KD_ROW_OK(d, N, p.status)) { __stcs(&out[d * kRowVec + t], rows[lr * kRowVec + t]); __stcs(&out[d * kRowVec + t + 8], rows[lr * kRowVec + t + 8]); }
                    // evicted cache rows among these four (rare): their terms, one warp per row, straight from the tile
                    for (unsigned gm = ((gone16 >> (4 * it)) & 0xfu) ? __ballot_sync(0xffffffffu, vis && d < 0 && seg_a + lr < len) & 0x01010101u : 0u; gm; gm &= gm - 1) {
                        const int glr = tile * kTileRows + it * 4 + ((__ffs(gm) - 1) >> 3);
                        warp_row_terms(reinterpret_cast<const uint2*>(rows + glr * kRowVec)[lane], true, inv_eps, raw, acc_g);
                    }
                }
                // The tile's only readers are this warp's lanes and their reads have returned (the stores
                // above consumed them), so the copy engine may overwrite it: a write after reads needs
                // execution order only, no proxy fence.
                __syncwarp();
                if (lane == 0) issue_tile(p.v_cache, p.new_v, u, len, B, N, sl, tile, rows_sa, mbar_sa);
            }
        }
        KD_STAMP(6);
        // ------------------------------------------------------------ the block rows of this CTA's range (requested before the
        // stores), every warp's sums into the tables, one barrier, and the delta and the next share are complete
        {
#pragma unroll
            for (int k = 0; k < kPreRows; ++k) {
                const int j = b_lo + warp + k * kFusedWarps;   // (warp-uniform conditions)
                if (block_row_evicted(j)) warp_row_terms(pre_e[k], true, inv_eps, raw, acc_g);
                if (next_share && j < b_hi) warp_row_terms(pre_n[k], true, inv_eps, raw, acc_n);
            }
            for (int j = b_lo + warp + kPreRows * kFusedWarps; j < b_hi; j += kFusedWarps) {   // ranges of more than 32 rows
                if (block_row_evicted(j))
                    warp_row_terms(reinterpret_cast<const uint2*>(blk_u + static_cast<size_t>(j) * kRowVec)[lane], true, inv_eps, raw, acc_g);
                if (next_share)
                    warp_row_terms(reinterpret_cast<const uint2*>(blk_n + static_cast<size_t>(j) * kRowVec)[lane], true, inv_eps, raw, acc_n);
            }
            // (both tables go through their two barriers together)
            {
                double2* rg = reinterpret_cast<double2*>(gone_tab + (warp & 7) * kHeadDim + 4 * lane);
                double2* rn = reinterpret_cast<double2*>(next_tab + (warp & 7) * kHeadDim + 4 * lane);
                if (warp < 8) {
                    rg[0] = make_double2(acc_g[0], acc_g[1]); rg[1] = make_double2(acc_g[2], acc_g[3]);
                    rn[0] = make_double2(acc_n[0], acc_n[1]); rn[1] = make_double2(acc_n[2], acc_n[3]);
                }
                __syncthreads();
                if (warp >= 8) {
                    double2 a = rg[0], b = rg[1];
                    rg[0] = make_double2(a.x + acc_g[0], a.y + acc_g[1]); rg[1] = make_double2(b.x + acc_g[2], b.y + acc_g[3]);
                    a = rn[0]; b = rn[1];
                    rn[0] = make_double2(a.x + acc_n[0], a.y + acc_n[1]); rn[1] = make_double2(b.x + acc_n[2], b.y + acc_n[3]);
                }
                __syncthreads();
            }
            if (tid < kHeadDim) {
                double gsum = 0.0, nsum = 0.0;
#pragma unroll
                for (int w = 0; w < 8; ++w) { gsum += gone_tab[w * kHeadDim + tid]; nsum += next_tab[w * kHeadDim + tid]; }
                p.anchor_delta[(static_cast<size_t>(u) * C + crank) * kHeadDim + tid] = (kOnePass ? partials[crank * kHeadDim + tid] : 0.0) - gsum;
                if (next_share) {
                    push_share(nsum);   // read by every CTA after the third cluster barrier (and by this one as its own share, a unit later)
                }
            }
        }
        KD_STAMP(7);
        // ------------------------------------------------------------ a4: V rows out, next unit's K rows in behind them
#pragma unroll 1
        for (int s = 0; s < kTilesPerWarp; ++s) {
            const int tile = warp + kFusedWarps * s;
            if (tile >= ntiles) break;
            if (min(rs, (tile + 1) * kTileRows) <= skip_local) continue;   // tile was not loaded
            mbar_wait(mbar_sa + 8 * tile, (parity >> s) & 1u, p.status);
            parity ^= 1u << s;
        }
        KD_STAMP(8);
        if (kRegRows > 0) {
            // The register-resident V rows must have ARRIVED, not merely been requested, before any peer may
            // overwrite their source: an empty asm statement that takes the words as inputs makes every one of
            // those loads complete in front of the barrier's arrive.
#pragma unroll
            for (int k = 0; k < kRegRows; ++k)
                asm volatile("" ::"r"(ra[k].x), "r"(ra[k].y), "r"(ra[k].z), "r"(ra[k].w),
                             "r"(rb[k].x), "r"(rb[k].y), "r"(rb[k].z), "r"(rb[k].w) : "memory");
        }
        cluster_sync_all();   // (3) every warp of the cluster holds the V rows it is responsible for
        KD_STAMP(9);
        if (kOnePass && un < p.U) {
            if (tid < kHeadDim) anchor_from_shares(folded_next, mu_buf + (cur ^ 1) * kHeadDim);
            __syncthreads();   // the next unit's anchor is complete before any warp scores with it
        }
        {
            uint4* out = p.v_cache + static_cast<size_t>(u) * N * kRowVec;
#pragma unroll
            for (int k = 0; k < kRegRows; ++k) {
                const int lr = rs + k * kGroups + g;
                if (lr < seg && lr >= skip_local) {
                    const int d = dst_of[lr];
                    if (d >= 0 && KD_ROW_OK(d, N, p.status)) { __stcs(&out[d * kRowVec + t], ra[k]); __stcs(&out[d * kRowVec + t + 8], rb[k]); }
                }
                if (lr < seg && un < p.U) {   // the next unit's K row takes the registers over
                    const uint4* row = concat_row(p.k_cache, p.new_k, un, seg_a + lr, len, B, N);
                    ra[k] = row[t]; rb[k] = row[t + 8];
                }
            }
            // V tiles out, the next unit's K tile in behind each, and -- one-pass steps -- the K tile that went in
            // behind the PREVIOUS V tile scored while this one's stores drain: the arithmetic runs under the copies
            const bool score_next = kOnePass && un < p.U;
            float2 w[8];
            float m = 0.f;
            if (score_next) {
                const float* mu_next = mu_buf + (cur ^ 1) * kHeadDim;
                load_anchor(mu_next, t, w);
                m = anchor_norm(mu_next, lane);
            }
            int prev = -1;   // this warp's previous tile slot: its K tile of the next unit is not scored yet
#pragma unroll 1
            for (int s = 0; s < kTilesPerWarp; ++s) {
                const int tile = warp + kFusedWarps * s;
                if (tile >= ntiles) break;
                if (min(rs, (tile + 1) * kTileRows) > skip_local) {
#pragma unroll
                    for (int it = 0; it < 4; ++it) {
                        const int lr = tile * kTileRows + it * 4 + sub;
                        if (lr < rs && lr >= skip_local) {
                            const int d = dst_of[lr];
                            if (d >= 0 && KD_ROW_OK(d, N, p.status)) { __stcs(&out[d * kRowVec + t], rows[lr * kRowVec + t]); __stcs(&out[d * kRowVec + t + 8], rows[lr * kRowVec + t + 8]); }
                        }
                    }
                    __syncwarp();
                }
                if (lane == 0 && un < p.U) issue_tile(p.k_cache, p.new_k, un, len, B, N, sl, tile, rows_sa, mbar_sa);
                if (score_next && prev >= 0) {
                    mbar_wait(mbar_sa + 8 * (warp + kFusedWarps * prev), (parity >> prev) & 1u, p.status);
                    parity ^= 1u << prev;
                    score_tile(rows, warp + kFusedWarps * prev, rs, t, sub, w, m, p.eps, keys + seg_a);
                }
                prev = s;
            }
            if (score_next) score_reg_rows(w, m);   // (their K rows were requested before the tiles: they are here by now)
            if (score_next && prev >= 0) {
                mbar_wait(mbar_sa + 8 * (warp + kFusedWarps * prev), (parity >> prev) & 1u, p.status);
                parity ^= 1u << prev;
                score_tile(rows, warp + kFusedWarps * prev, rs, t, sub, w, m, p.eps, keys + seg_a);
            }
        }
        KD_STAMP(10);
        if (kOnePass && un < p.U) {
            tiles_scored = true;
            cur ^= 1;
        }
        KD_STAMP(11);
        __syncthreads();   // dst_of is free for the next unit
        KD_STAMP(12);
    }
    cluster_sync_all();   // no CTA leaves while a peer may still address its shared memory
    KD_STAMP(13);
    KD_STAMP_FLUSH;
}

}  // namespace kd
