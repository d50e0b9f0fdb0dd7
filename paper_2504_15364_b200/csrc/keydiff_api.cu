// Host side of the KeyDiff eviction-step library: context, argument validation, launch
// configuration and the extern "C" entry points declared in include/keydiff.h.
#include "../../include/keydiff.h"

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <mutex>
#include <new>

#include "common.cuh"
#include "staged_kernels.cuh"
#include "fused_kernel.cuh"
#include "slot_kernel.cuh"

namespace {

thread_local int g_last_cuda_error = 0;

inline bool cuda_ok(cudaError_t e) {
    if (e == cudaSuccess) return true;
    g_last_cuda_error = static_cast<int>(e);
    return false;
}
#define KD_CUDA(call) do { if (!cuda_ok(call)) return KEYDIFF_ERR_CUDA; } while (0)

constexpr float kDefaultEps = 1e-8f;

// Launch-tuning aids (named in include/keydiff.h): read from the environment ONCE, by keydiff_create; a step
// never looks at the environment.  A value < 0 means "not set".
int env_int(const char* name) {
    const char* v = std::getenv(name);
    return (v && *v) ? std::atoi(v) : -1;
}

// Test hook (keydiff_debug_fail_alloc): the n-th device allocation from now on fails once.
int g_fail_alloc_countdown = 0;
cudaError_t kd_malloc(void** p, size_t bytes) {
    if (g_fail_alloc_countdown > 0 && --g_fail_alloc_countdown == 0) { *p = nullptr; return cudaErrorMemoryAllocation; }
    return cudaMalloc(p, bytes);
}
template <typename T> cudaError_t kd_malloc(T** p, size_t bytes) { return kd_malloc(reinterpret_cast<void**>(p), bytes); }
constexpr int kMaxSelectSmem = 200 * 1024;   // score keys of one unit must fit one CTA

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

struct keydiff_ctx {
    keydiff_config cfg;
    int U = 0;            // independent units = n_layers * batch * n_kv_heads
    int nmax = 0;         // N + max_block
    int len = 0;          // tokens currently cached (same for every unit)
    int splits = 1;       // row slices per unit in the staged anchor/score kernels
    int path = KEYDIFF_PATH_STAGED;
    int cluster = 1;            // fused path: CTAs per cluster
    int fused_smem_rows = 0;    // fused path: slice rows resident in shared memory
    int fused_nkeys = 0;        // fused path: key-table capacity
    int fused_smem_bytes = 0;
    int fused_max_clusters = 0; // co-resident clusters (grid = min(U, this) * cluster)
    int fused_reg_rows = 0;     // kernel instance: rows per row group kept in registers
    bool slot_stream = false;   // slot reuse: the streaming kernel serves the step (cluster, fused_nkeys,
    int slot_ring_tiles = 0;    //   fused_smem_bytes, fused_max_clusters describe it)
    int slot_nwords = 0;
    int sm_count = 0;           // SMs of the ctx's device
    int tune_cluster = -1, tune_stagger_ns = -1, tune_late_ns = -1, tune_max_clusters = -1;   // KEYDIFF_* tuning aids as keydiff_create read them
    // running anchor of the fused path: sum of k/||k|| over the cached rows, per unit
    bool incremental = true;    // use it (one-pass kernel) when it is valid
    bool anchor_valid = false;  // the buffers describe the cache as the last evicting step left it
    int anchor_par = 0;         // which of the two sum buffers the next step reads
    int steps_since_full = 0;   // one-pass steps since the anchor was last recomputed from all rows
    double* anchor_sum[2] = {nullptr, nullptr};   // [U][128]
    double* anchor_delta = nullptr;               // [U][cluster][128]
    float eps = kDefaultEps;
    // device scratch
    double* partial = nullptr;        // [U][splits][128]
    float* norms = nullptr;           // [U][nmax]
    float* scores = nullptr;          // [U][nmax]
    int32_t* kept_idx = nullptr;      // [U][N]
    int32_t* first_evicted = nullptr; // [U]
    int32_t* status = nullptr;        // [1]
    unsigned long long* moved_rows = nullptr;   // [1] cumulative count of rows that changed position
    // unordered slot reuse: token position held by every slot, and the position of the next new token
    int32_t* pos = nullptr;           // [U][N]
    long long next_pos = 0;
    bool pos_stale = true;            // pos must be reset to the identity before the next step uses it
    // keydiff_evict_host only: two sets of staging buffers [U][max_block][128] bf16 filled on a copy stream
    // of the ctx, so that the block of step i+1 crosses the bus while the kernels of step i run
    void* stage_k[2] = {nullptr, nullptr};
    void* stage_v[2] = {nullptr, nullptr};
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_copied[2] = {nullptr, nullptr};   // the set's block has arrived
    cudaEvent_t ev_consumed[2] = {nullptr, nullptr}; // the step that read the set has finished
    bool consumed_recorded[2] = {false, false};
    int stage_next = 0;
    int32_t* kept_mirror = nullptr;   // set by keydiff_evict_host around its step: the fused kernels also write the
                                      // kept-index list there (the caller's pinned buffer), so no copy follows
};

namespace {

void free_scratch(keydiff_ctx* c) {
    cudaFree(c->partial); cudaFree(c->norms); cudaFree(c->scores); cudaFree(c->kept_idx);
    cudaFree(c->first_evicted); cudaFree(c->status); cudaFree(c->moved_rows);
    for (int b = 0; b < 2; ++b) {
        cudaFree(c->stage_k[b]); cudaFree(c->stage_v[b]);
        if (c->ev_copied[b]) cudaEventDestroy(c->ev_copied[b]);
        if (c->ev_consumed[b]) cudaEventDestroy(c->ev_consumed[b]);
    }
    if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
    cudaFree(c->anchor_sum[0]); cudaFree(c->anchor_sum[1]); cudaFree(c->anchor_delta); cudaFree(c->pos);
}

int check_step_args(const keydiff_ctx* ctx, const void* k_cache, const void* v_cache,
                    const void* new_k, const void* new_v, int32_t N, int32_t B, int32_t H, int32_t d) {
    if (!ctx || !k_cache || !v_cache || !new_k || !new_v) return KEYDIFF_ERR_INVALID_ARG;
    if (N != ctx->cfg.budget || H != ctx->cfg.n_kv_heads || d != ctx->cfg.head_dim) return KEYDIFF_ERR_INVALID_ARG;
    if (B < 1 || B > ctx->cfg.max_block) return KEYDIFF_ERR_INVALID_ARG;
    if (!aligned16(k_cache) || !aligned16(v_cache) || !aligned16(new_k) || !aligned16(new_v)) return KEYDIFF_ERR_INVALID_ARG;
    if (k_cache == v_cache || k_cache == new_k || v_cache == new_v) return KEYDIFF_ERR_INVALID_ARG;
    int dev = -1;
    KD_CUDA(cudaGetDevice(&dev));
    if (dev != ctx->cfg.device) return KEYDIFF_ERR_STATE;   // the ctx's device must be current
    return KEYDIFF_OK;
}

inline int prop_sm_count(const keydiff_ctx* c) { return c->sm_count > 0 ? c->sm_count : 148; }
inline bool slot_reuse(const keydiff_ctx* c) { return c->cfg.compaction == KEYDIFF_COMPACT_SLOT_REUSE; }

using FusedKernel = void (*)(kd::FusedParams);

// Kernel instance for `reg_rows` register-resident rows per row group (rounded up to one that is
// built); one_pass = the variant that takes the anchor from the running sum; few_pre = the variant that holds one
// block row per warp and kind across the K stores instead of four (one-pass kernels only).
template <bool kOnePass, int kPre>
FusedKernel fused_instance_of(int reg_rows, int* built) {
    using namespace kd;
    if (reg_rows <= 0) { *built = 0; return fused_evict_kernel<0, kOnePass, kPre>; }
    if (reg_rows <= 2) { *built = 2; return fused_evict_kernel<2, kOnePass, kPre>; }
    if (reg_rows <= 4) { *built = 4; return fused_evict_kernel<4, kOnePass, kPre>; }
    if (reg_rows <= 5) { *built = 5; return fused_evict_kernel<5, kOnePass, kPre>; }
    *built = 6; return fused_evict_kernel<6, kOnePass, kPre>;
}
FusedKernel fused_instance(int reg_rows, int* built, bool one_pass = false, bool few_pre = false) {
    if (!one_pass) return fused_instance_of<false, 4>(reg_rows, built);
    return few_pre ? fused_instance_of<true, 1>(reg_rows, built) : fused_instance_of<true, 4>(reg_rows, built);
}

// Co-resident clusters of `C` CTAs of the kernel `kern` with `smem` bytes each.
template <typename Kernel>
int max_active_clusters(Kernel kern, int C, int smem, int sm_count) {
    using namespace kd;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return 0;
    if (C > 8 && cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) return 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(C * sm_count);
    cfg.blockDim = dim3(kFusedThreads);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
    return n;
}

// Choose the cluster size and shared-memory split of the fused kernel for units of up to nmax
// rows; returns false if no cluster can hold a unit on chip.  Every cluster size from 1 to 16 is
// tried: how many clusters the device holds at once depends on how the SMs are grouped (on a B200
// 15 clusters fit both at 8 and at 9 CTAs, i.e. 120 or 135 SMs), and the estimated step time
//   ceil(U / clusters) * (fixed cost per unit + cost per slice row * slice rows)
// picks the winner (constants from per-phase timings of the kernel on a B200).
bool plan_fused(keydiff_ctx* c, int sm_count) {
    using namespace kd;
    constexpr double kUnitFixedUs = 10.0, kRowUs = 0.0165, kManyRegRowsUs = 4.5;   // (more than 4 register rows: spills)
    const int forced = c->tune_cluster;
    double best = 0.0;
    bool found = false;
    for (int C = 1; C <= kMaxCluster; ++C) {
        if (forced > 0 && C != forced) continue;
        const int per_cta = ((c->nmax + C - 1) / C + 3) & ~3;        // slices are multiples of 4 rows
        const int nkeys = C * per_cta;
        int sr = std::min(kMaxTiles * kTileRows, (per_cta + kTileRows - 1) / kTileRows * kTileRows);
        while (sr > 0 && fused_layout(sr, nkeys, C).total > kSmemLimit) sr -= kTileRows;
        if (sr <= 0) break;                                          // the key table alone does not fit
        if (sr + kMaxRegRows * kGroups < per_cta) continue;          // slice too long for this cluster size
        const int smem = fused_layout(sr, nkeys, C).total;
        int reg_rows = 0;
        const FusedKernel kern = fused_instance((std::max(0, per_cta - sr) + kGroups - 1) / kGroups, &reg_rows);
        const int clusters = max_active_clusters(kern, C, smem, sm_count);
        if (clusters < 1) continue;
        const int used = std::min(c->U, clusters);
        const double est = static_cast<double>((c->U + used - 1) / used) *
                           (kUnitFixedUs + kRowUs * per_cta + (reg_rows > 4 ? kManyRegRowsUs : 0.0));
        if (!found || est < 0.95 * best) {   // a larger cluster has to pay for its extra barrier traffic
            found = true; best = est;
            c->cluster = C; c->fused_smem_rows = sr; c->fused_nkeys = nkeys; c->fused_smem_bytes = smem;
            c->fused_max_clusters = clusters; c->fused_reg_rows = reg_rows;
        }
    }
    if (!found) return false;
    // the attributes of the chosen instance (the loop may have left another size's values behind)
    int built = 0;
    return max_active_clusters(fused_instance(c->fused_reg_rows, &built, false), c->cluster, c->fused_smem_bytes, sm_count) >= 1 &&
           max_active_clusters(fused_instance(c->fused_reg_rows, &built, true, false), c->cluster, c->fused_smem_bytes, sm_count) >= 1 &&
           max_active_clusters(fused_instance(c->fused_reg_rows, &built, true, true), c->cluster, c->fused_smem_bytes, sm_count) >= 1;
}

// Slot reuse: cluster size and ring of the streaming kernel for units of up to nmax rows; false if it
// cannot serve the configuration (then the resident kernel or the staged path does).  Nothing has to
// stay on chip, so small clusters are possible and many units are in flight; the estimate
//   ceil(U / clusters) * (fixed cost per unit + cost per slice row * slice rows)
// picks the size (constants from per-phase timings on a B200: anchor, selection, lists and barriers are
// a fixed cost, the stream runs at the pace of one SM's share of the HBM bandwidth).
bool plan_slot_stream(keydiff_ctx* c, int sm_count) {
    using namespace kd;
    if (c->cfg.max_block > kSlotMaxBlock) return false;
    const int forced = c->tune_cluster;
    const int nwords = (c->nmax + 31) / 32;
    double best = 0.0;
    bool found = false;
    for (int C = 1; C <= kMaxCluster; ++C) {
        if (forced > 0 && C != forced) continue;
        const int per_cta = ((c->nmax + C - 1) / C + kTileRows - 1) / kTileRows * kTileRows;
        const int nkeys = C * per_cta;
        int ring = 3 * kFusedWarps;   // up to three tiles per warp in flight
        while (ring > 0 && slot_layout(ring, nkeys, nwords, c->cfg.max_block).total > kSmemLimit) ring -= kFusedWarps;
        if (ring <= 0) continue;
        const int smem = slot_layout(ring, nkeys, nwords, c->cfg.max_block).total;
        const int clusters = max_active_clusters(slot_evict_kernel, C, smem, sm_count);
        if (clusters < 1) continue;
        const int used = std::min(c->U, clusters);
        const double row_us = 256.0 / (6.0e6 / std::min(sm_count, used * C));   // one SM's share of ~6 TB/s, in bytes per us
        const double est = static_cast<double>((c->U + used - 1) / used) * ((C > 1 ? 11.0 : 9.0) + std::max(row_us, 0.0045) * per_cta);
        if (!found || est < best) {
            found = true; best = est;
            c->cluster = C; c->fused_nkeys = nkeys; c->fused_smem_bytes = smem; c->fused_max_clusters = clusters;
            c->slot_ring_tiles = ring; c->slot_nwords = nwords;
        }
    }
    if (!found) return false;
    return max_active_clusters(slot_evict_kernel, c->cluster, c->fused_smem_bytes, sm_count) >= 1;
}

int launch_slot_stream(keydiff_ctx* c, uint4* kc, uint4* vc, const uint4* nk, const uint4* nv, int B, cudaStream_t st) {
    using namespace kd;
    const int N = c->cfg.budget, n = c->len + B;
    if (!(c->incremental && c->anchor_valid && c->steps_since_full < 1024)) {
        // the running sum of the cached rows, rebuilt from all of them: first evicting step, after appends,
        // set_len / reset, periodically against rounding drift, and every step when the caller asked for it
        const int rows_per_split = (c->len + c->splits - 1) / c->splits;
        anchor_partial_kernel<<<dim3(c->splits, c->U), kStagedThreads, 0, st>>>(kc, nk, c->len, 0, N, c->eps, rows_per_split, c->nmax,
                                                                               c->partial, c->norms, c->cfg.anchor_mode == KEYDIFF_ANCHOR_RAW_MEAN);
        anchor_fold_kernel<<<c->U, kHeadDim, 0, st>>>(c->partial, c->splits, c->anchor_sum[c->anchor_par], c->anchor_delta, c->cluster);
        c->steps_since_full = 0;
    } else {
        ++c->steps_since_full;
    }
    SlotParams p;
    p.k_cache = kc; p.v_cache = vc; p.new_k = nk; p.new_v = nv;
    p.len = c->len; p.B = B; p.N = N; p.U = c->U; p.eps = c->eps;
    p.cluster = c->cluster;
    p.rows_per_cta = ((n + c->cluster - 1) / c->cluster + kTileRows - 1) / kTileRows * kTileRows;
    p.ring_tiles = c->slot_ring_tiles; p.nkeys = c->fused_nkeys; p.nwords = c->slot_nwords; p.nmax = c->nmax;
    p.max_block = c->cfg.max_block;
    p.scores = c->scores; p.kept_idx = c->kept_idx; p.first_evicted = c->first_evicted;
    p.moved_rows = c->moved_rows; p.status = c->status;
    p.anchor_in = c->anchor_sum[c->anchor_par];
    p.anchor_out = c->anchor_sum[c->anchor_par ^ 1];
    p.anchor_delta = c->anchor_delta;
    p.raw_anchor = c->cfg.anchor_mode == KEYDIFF_ANCHOR_RAW_MEAN;
    p.window = c->cfg.recent_window;
    p.pos = c->pos; p.next_pos = static_cast<int>(c->next_pos);
    p.kept_mirror = c->kept_mirror;
    const int nclusters = std::min(c->U, c->fused_max_clusters);
    // Start-up stagger: clusters launched together stream together and then select together, leaving HBM
    // idle in between.  When every cluster serves at least three units, starting cluster c a little later
    // than cluster c-1 (about half a unit's duration over all of them) spreads the phases; with fewer
    // units per cluster the delay would only postpone the end (sweep on a B200: 896 units of 4352 rows
    // gain 12 %, 256 units of 8320 rows lose 3 %).
    p.stagger_ns = 0;
    p.late_ns = 0;
    {
        const double share = 6500.0 / std::min(prop_sm_count(c), nclusters * c->cluster);   // bytes per ns for one SM
        const double unit_ns = 9000.0 + static_cast<double>(p.rows_per_cta) * kRowBytes / share;
        if (nclusters > 1 && c->U >= 3 * nclusters) {
            p.stagger_ns = static_cast<unsigned>(0.55 * unit_ns / nclusters);
        } else if (c->U > nclusters && c->U % nclusters != 0) {
            // Two rounds, the second one partial: the clusters with a single unit start half a unit late, so that
            // they stream while the others are between their two streams (sweep on a B200: best at 0.4-0.6 of a
            // unit's duration; 256 units of 8320 rows gain 5 %, 224 units of 2176 rows 6 %)
            p.late_ns = static_cast<unsigned>(0.5 * unit_ns);
        }
    }
    if (c->tune_stagger_ns >= 0) p.stagger_ns = static_cast<unsigned>(c->tune_stagger_ns);
    if (c->tune_late_ns >= 0) p.late_ns = static_cast<unsigned>(c->tune_late_ns);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(nclusters * c->cluster);
    cfg.blockDim = dim3(kFusedThreads);
    cfg.dynamicSmemBytes = c->fused_smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = c->cluster; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    KD_CUDA(cudaLaunchKernelEx(&cfg, slot_evict_kernel, p));
    KD_CUDA(cudaGetLastError());
    c->anchor_par ^= 1;
    c->anchor_valid = true;
    return KEYDIFF_OK;
}

int launch_fused(keydiff_ctx* c, uint4* kc, uint4* vc, const uint4* nk, const uint4* nv, int B, cudaStream_t st) {
    if (c->slot_stream) return launch_slot_stream(c, kc, vc, nk, nv, B, st);
    using namespace kd;
    FusedParams p;
    p.k_cache = kc; p.v_cache = vc; p.new_k = nk; p.new_v = nv;
    p.len = c->len; p.B = B; p.N = c->cfg.budget; p.U = c->U; p.eps = c->eps;
    p.cluster = c->cluster;
    p.rows_per_cta = ((c->len + B + c->cluster - 1) / c->cluster + 3) & ~3;
    p.smem_rows = c->fused_smem_rows; p.nkeys = c->fused_nkeys; p.nmax = c->nmax;
    p.scores = c->scores; p.kept_idx = c->kept_idx; p.first_evicted = c->first_evicted;
    p.moved_rows = c->moved_rows; p.status = c->status;
    // The one-pass kernel needs the running anchor of the cache as it stands; every 1024 steps the
    // anchor is recomputed from all rows anyway, which sheds whatever rounding drift has built up.
    const bool one_pass = c->incremental && c->anchor_valid && c->steps_since_full < 1024;
    p.anchor_in = c->anchor_sum[c->anchor_par];
    p.anchor_out = c->anchor_sum[c->anchor_par ^ 1];
    p.anchor_delta = c->anchor_delta;
    p.raw_anchor = c->cfg.anchor_mode == KEYDIFF_ANCHOR_RAW_MEAN;
    p.window = c->cfg.recent_window;
    p.kept_mirror = c->kept_mirror;
    int nclusters = std::min(c->U, c->fused_max_clusters);
    if (c->tune_max_clusters > 0) nclusters = std::min(nclusters, c->tune_max_clusters);
    // Start-up stagger: somewhat less than one unit's duration spread evenly over the co-resident
    // clusters.  A unit moves 4 slices (K in, K out, V in, V out) per SM at roughly 60 GB/s per SM when
    // the other SMs are busy too, plus a few microseconds of arithmetic and barriers (a sweep of the
    // delay on a B200 put the best value at 0.7-0.95 of unit time / clusters for the large workloads).
    p.stagger_ns = 0;
    if (nclusters > 1 && c->U > nclusters) {
        const double unit_ns = 4.0 * p.rows_per_cta * kRowBytes / 60.0 + 6000.0;
        p.stagger_ns = static_cast<unsigned>(unit_ns / nclusters);
    }
    if (c->tune_stagger_ns >= 0) p.stagger_ns = static_cast<unsigned>(c->tune_stagger_ns);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(nclusters * c->cluster);
    cfg.blockDim = dim3(kFusedThreads);
    cfg.dynamicSmemBytes = c->fused_smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = c->cluster; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int built = 0;
    const bool few_pre = B <= 16 * c->cluster;   // a CTA's share of the block: at most one row per warp
    KD_CUDA(cudaLaunchKernelEx(&cfg, fused_instance(c->fused_reg_rows, &built, one_pass, few_pre), p));
    c->anchor_par ^= 1;
    c->anchor_valid = true;
    c->steps_since_full = one_pass ? c->steps_since_full + 1 : 0;
    return KEYDIFF_OK;
}

int launch_staged(keydiff_ctx* c, uint4* kc, uint4* vc, const uint4* nk, const uint4* nv, int B, cudaStream_t st) {
    using namespace kd;
    const int N = c->cfg.budget, n = c->len + B, U = c->U;
    const int rows_per_split = (n + c->splits - 1) / c->splits;
    const dim3 grid(c->splits, U);
    anchor_partial_kernel<<<grid, kStagedThreads, 0, st>>>(kc, nk, c->len, B, N, c->eps, rows_per_split, c->nmax,
                                                           c->partial, c->norms, c->cfg.anchor_mode == KEYDIFF_ANCHOR_RAW_MEAN);
    score_kernel<<<grid, kStagedThreads, 0, st>>>(kc, nk, c->len, B, N, c->eps, rows_per_split, c->nmax,
                                                  c->partial, c->norms, c->scores);
    select_kernel<<<U, kSelectThreads, static_cast<size_t>(n) * 4, st>>>(c->scores, n, N, c->nmax, c->len, c->kept_idx,
                                                                          c->first_evicted, c->moved_rows, c->cfg.recent_window,
                                                                          slot_reuse(c) ? c->pos : nullptr, static_cast<int>(c->next_pos));
    if (slot_reuse(c))
        slot_place_kernel<<<U, kCompactThreads, static_cast<size_t>(B) * 8, st>>>(kc, vc, nk, nv, c->len, B, N, c->kept_idx, c->pos,
                                                                                  static_cast<int>(c->next_pos), c->moved_rows);
    else
        compact_kernel<<<dim3(2, U), kCompactThreads, 0, st>>>(kc, vc, nk, nv, c->len, B, N, c->kept_idx, c->first_evicted, c->status);
    KD_CUDA(cudaGetLastError());
    return KEYDIFF_OK;
}

}  // namespace

namespace {
int create_impl(const keydiff_config* cfg, keydiff_ctx** out) {
    if (!cfg || !out) return KEYDIFF_ERR_INVALID_ARG;
    if (cfg->n_layers < 1 || cfg->batch < 1 || cfg->n_kv_heads < 1 || cfg->budget < 1 || cfg->max_block < 1 ||
        cfg->device < 0 || cfg->eps < 0.f)
        return KEYDIFF_ERR_INVALID_ARG;
    if (cfg->path != KEYDIFF_PATH_AUTO && cfg->path != KEYDIFF_PATH_STAGED && cfg->path != KEYDIFF_PATH_FUSED)
        return KEYDIFF_ERR_INVALID_ARG;
    if (cfg->anchor_mode != KEYDIFF_ANCHOR_NORMALISED && cfg->anchor_mode != KEYDIFF_ANCHOR_RAW_MEAN) return KEYDIFF_ERR_INVALID_ARG;
    if (cfg->recent_window < 0 || cfg->recent_window > cfg->budget) return KEYDIFF_ERR_INVALID_ARG;
    if (cfg->compaction != KEYDIFF_COMPACT_ORDERED && cfg->compaction != KEYDIFF_COMPACT_SLOT_REUSE) return KEYDIFF_ERR_INVALID_ARG;
    if (cfg->dtype != KEYDIFF_BF16 || cfg->head_dim != kd::kHeadDim) return KEYDIFF_ERR_UNSUPPORTED;
    const long long U = 1LL * cfg->n_layers * cfg->batch * cfg->n_kv_heads;
    const long long nmax = 1LL * cfg->budget + cfg->max_block;
    if (U > 65535 || nmax > (1 << 30)) return KEYDIFF_ERR_UNSUPPORTED;   // gridDim.y limit of the staged kernels
    if (nmax * 4 > kMaxSelectSmem) return KEYDIFF_ERR_UNSUPPORTED;
    if (cfg->compaction == KEYDIFF_COMPACT_SLOT_REUSE && 8LL * cfg->max_block > kMaxSelectSmem) return KEYDIFF_ERR_UNSUPPORTED;

    int count = 0;
    KD_CUDA(cudaGetDeviceCount(&count));
    if (cfg->device >= count) return KEYDIFF_ERR_INVALID_ARG;
    cudaDeviceProp prop;
    KD_CUDA(cudaGetDeviceProperties(&prop, cfg->device));
    if (prop.major != 10) return KEYDIFF_ERR_UNSUPPORTED;   // built for sm_100a only; no fallback

    int prev = -1;
    KD_CUDA(cudaGetDevice(&prev));
    KD_CUDA(cudaSetDevice(cfg->device));

    keydiff_ctx* c = new (std::nothrow) keydiff_ctx();
    if (!c) { cudaSetDevice(prev); return KEYDIFF_ERR_ALLOC; }
    c->cfg = *cfg;
    c->U = static_cast<int>(U);
    c->nmax = static_cast<int>(nmax);
    c->eps = cfg->eps > 0.f ? cfg->eps : kDefaultEps;
    c->sm_count = prop.multiProcessorCount;
    c->tune_cluster = env_int("KEYDIFF_CLUSTER_SIZE");
    c->tune_stagger_ns = env_int("KEYDIFF_STAGGER_NS");
    c->tune_late_ns = env_int("KEYDIFF_LATE_NS");
    c->tune_max_clusters = env_int("KEYDIFF_MAX_CLUSTERS");
    c->path = KEYDIFF_PATH_STAGED;
    // enough CTAs to fill 148 SMs a few times over, but at least 64 rows per slice
    const int want = (4 * prop.multiProcessorCount + c->U - 1) / c->U;
    c->splits = std::max(1, std::min({want, (c->nmax + 63) / 64, 64}));

    bool ok = true;
    ok = ok && kd_malloc(&c->partial, sizeof(double) * c->U * c->splits * kd::kHeadDim) == cudaSuccess;
    ok = ok && kd_malloc(&c->norms, sizeof(float) * U * nmax) == cudaSuccess;
    ok = ok && kd_malloc(&c->scores, sizeof(float) * U * nmax) == cudaSuccess;
    ok = ok && kd_malloc(&c->kept_idx, sizeof(int32_t) * U * cfg->budget) == cudaSuccess;
    ok = ok && kd_malloc(&c->first_evicted, sizeof(int32_t) * U) == cudaSuccess;
    ok = ok && kd_malloc(&c->status, sizeof(int32_t)) == cudaSuccess;
    ok = ok && kd_malloc(&c->moved_rows, sizeof(unsigned long long)) == cudaSuccess;
    if (ok) {
        ok = cudaMemset(c->scores, 0, sizeof(float) * U * nmax) == cudaSuccess &&
             cudaMemset(c->kept_idx, 0, sizeof(int32_t) * U * cfg->budget) == cudaSuccess &&
             cudaMemset(c->first_evicted, 0, sizeof(int32_t) * U) == cudaSuccess &&
             cudaMemset(c->status, 0, sizeof(int32_t)) == cudaSuccess &&
             cudaMemset(c->moved_rows, 0, sizeof(unsigned long long)) == cudaSuccess;
    }
    if (ok) {
        ok = cudaFuncSetAttribute(kd::select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  kMaxSelectSmem) == cudaSuccess;
    }
    if (ok && cfg->compaction == KEYDIFF_COMPACT_SLOT_REUSE) {
        ok = kd_malloc(&c->pos, sizeof(int32_t) * U * cfg->budget) == cudaSuccess &&
             cudaMemset(c->pos, 0, sizeof(int32_t) * U * cfg->budget) == cudaSuccess &&
             cudaFuncSetAttribute(kd::slot_place_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  std::max(48 * 1024, 8 * cfg->max_block)) == cudaSuccess;
    }
    if (ok) ok = cudaDeviceSynchronize() == cudaSuccess;
    if (ok && cfg->path != KEYDIFF_PATH_STAGED) {
        // slot reuse is served by the streaming kernel (or, where that cannot hold a unit's keys, by the staged path)
        c->slot_stream = slot_reuse(c) && plan_slot_stream(c, prop.multiProcessorCount);
        if (c->slot_stream || (!slot_reuse(c) && plan_fused(c, prop.multiProcessorCount))) {
            c->path = KEYDIFF_PATH_FUSED;
            const size_t sum_bytes = sizeof(double) * U * kd::kHeadDim;
            ok = kd_malloc(&c->anchor_sum[0], sum_bytes) == cudaSuccess && kd_malloc(&c->anchor_sum[1], sum_bytes) == cudaSuccess &&
                 kd_malloc(&c->anchor_delta, sizeof(double) * U * c->cluster * kd::kHeadDim) == cudaSuccess &&
                 cudaMemset(c->anchor_sum[0], 0, sum_bytes) == cudaSuccess && cudaMemset(c->anchor_sum[1], 0, sum_bytes) == cudaSuccess &&
                 cudaMemset(c->anchor_delta, 0, sizeof(double) * U * c->cluster * kd::kHeadDim) == cudaSuccess &&
                 cudaDeviceSynchronize() == cudaSuccess;
        } else if (cfg->path == KEYDIFF_PATH_FUSED) {
            free_scratch(c);
            delete c;
            cudaSetDevice(prev);
            return KEYDIFF_ERR_UNSUPPORTED;
        }
    }
    if (!ok) {
        g_last_cuda_error = static_cast<int>(cudaGetLastError());
        free_scratch(c);
        delete c;
        cudaSetDevice(prev);
        return KEYDIFF_ERR_ALLOC;
    }
    cudaSetDevice(prev);
    *out = c;
    return KEYDIFF_OK;
}
}  // namespace

extern "C" {

int keydiff_create(const keydiff_config* cfg, keydiff_ctx** out) {
    const int rc = create_impl(cfg, out);
    g_fail_alloc_countdown = 0;   // the test hook serves one keydiff_create
    return rc;
}

int keydiff_evict(keydiff_ctx* ctx, void* k_cache, void* v_cache, const void* new_k, const void* new_v,
                  int32_t budget_N, int32_t block_B, int32_t n_kv_heads, int32_t head_dim, void* stream) {
    const int rc = check_step_args(ctx, k_cache, v_cache, new_k, new_v, budget_N, block_B, n_kv_heads, head_dim);
    if (rc != KEYDIFF_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint4* kc = static_cast<uint4*>(k_cache);
    uint4* vc = static_cast<uint4*>(v_cache);
    const uint4* nk = static_cast<const uint4*>(new_k);
    const uint4* nv = static_cast<const uint4*>(new_v);
    const int N = ctx->cfg.budget, n = ctx->len + block_B;
    if (slot_reuse(ctx)) {
        if (ctx->next_pos + block_B > 0x7fffffffLL) return KEYDIFF_ERR_STATE;   // positions are int32
        if (ctx->pos_stale) {
            // the cache as the caller declared it: slot s holds token s
            const int total = ctx->U * N;
            kd::pos_iota_kernel<<<(total + 255) / 256, 256, 0, st>>>(ctx->pos, N, total);
            ctx->pos_stale = false;
        }
    }
    if (n <= N) {
        // Sec. 2.3: the budget is not exceeded, nothing is evicted
        const int threads = 256;
        const dim3 grid((block_B * kd::kRowVec + threads - 1) / threads, ctx->U, 2);
        kd::append_kernel<<<grid, threads, 0, st>>>(kc, vc, nk, nv, ctx->len, block_B, N);
        if (slot_reuse(ctx))
            kd::pos_append_kernel<<<dim3((block_B + threads - 1) / threads, ctx->U), threads, 0, st>>>(
                ctx->pos, ctx->len, block_B, N, static_cast<int>(ctx->next_pos));
        KD_CUDA(cudaGetLastError());
        ctx->len = n;
        ctx->next_pos += block_B;
        ctx->anchor_valid = false;   // the appended rows are not in the running anchor
        return KEYDIFF_OK;
    }
    const int lrc = ctx->path == KEYDIFF_PATH_FUSED ? launch_fused(ctx, kc, vc, nk, nv, block_B, st)
                                                    : launch_staged(ctx, kc, vc, nk, nv, block_B, st);
    if (lrc != KEYDIFF_OK) return lrc;
    ctx->len = N;
    ctx->next_pos += block_B;
    return KEYDIFF_OK;
}

int keydiff_evict_host(keydiff_ctx* ctx, void* k_cache, void* v_cache, const void* new_k_host, const void* new_v_host,
                       int32_t budget_N, int32_t block_B, int32_t n_kv_heads, int32_t head_dim,
                       int32_t* kept_idx_host, int32_t* status_host, void* stream) {
    if (!ctx || !new_k_host || !new_v_host) return KEYDIFF_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!ctx->copy_stream) {
        const size_t bytes = static_cast<size_t>(ctx->U) * ctx->cfg.max_block * kd::kRowBytes;
        bool ok = cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
        for (int b = 0; b < 2 && ok; ++b)
            ok = cudaMalloc(&ctx->stage_k[b], bytes) == cudaSuccess && cudaMalloc(&ctx->stage_v[b], bytes) == cudaSuccess &&
                 cudaEventCreateWithFlags(&ctx->ev_copied[b], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&ctx->ev_consumed[b], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) {
            g_last_cuda_error = static_cast<int>(cudaGetLastError());
            for (int b = 0; b < 2; ++b) {
                cudaFree(ctx->stage_k[b]); cudaFree(ctx->stage_v[b]); ctx->stage_k[b] = ctx->stage_v[b] = nullptr;
                if (ctx->ev_copied[b]) { cudaEventDestroy(ctx->ev_copied[b]); ctx->ev_copied[b] = nullptr; }
                if (ctx->ev_consumed[b]) { cudaEventDestroy(ctx->ev_consumed[b]); ctx->ev_consumed[b] = nullptr; }
            }
            if (ctx->copy_stream) { cudaStreamDestroy(ctx->copy_stream); ctx->copy_stream = nullptr; }
            return KEYDIFF_ERR_ALLOC;
        }
    }
    const int b = ctx->stage_next;
    const int rc = check_step_args(ctx, k_cache, v_cache, ctx->stage_k[b], ctx->stage_v[b], budget_N, block_B, n_kv_heads, head_dim);
    if (rc != KEYDIFF_OK) return rc;
    const size_t bytes = static_cast<size_t>(ctx->U) * block_B * kd::kRowBytes;
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    KD_CUDA(cudaStreamIsCapturing(st, &capturing));
    if (capturing == cudaStreamCaptureStatusNone) {
        // the copy does not wait for what is queued on `st`: only for the step that last read this set
        if (ctx->consumed_recorded[b]) KD_CUDA(cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_consumed[b], 0));
        KD_CUDA(cudaMemcpyAsync(ctx->stage_k[b], new_k_host, bytes, cudaMemcpyHostToDevice, ctx->copy_stream));
        KD_CUDA(cudaMemcpyAsync(ctx->stage_v[b], new_v_host, bytes, cudaMemcpyHostToDevice, ctx->copy_stream));
        KD_CUDA(cudaEventRecord(ctx->ev_copied[b], ctx->copy_stream));
        KD_CUDA(cudaStreamWaitEvent(st, ctx->ev_copied[b], 0));
    } else {
        // inside a stream capture everything stays on the captured stream
        KD_CUDA(cudaMemcpyAsync(ctx->stage_k[b], new_k_host, bytes, cudaMemcpyHostToDevice, st));
        KD_CUDA(cudaMemcpyAsync(ctx->stage_v[b], new_v_host, bytes, cudaMemcpyHostToDevice, st));
    }
    // Pinned host memory has a device alias: on the fused path an evicting step writes the kept-index list
    // there itself, as it writes it to scratch, so the list crosses the bus during the step
    bool mirrored = false;
    if (kept_idx_host && ctx->path == KEYDIFF_PATH_FUSED && ctx->len + block_B > ctx->cfg.budget) {
        cudaPointerAttributes attr;
        if (cudaPointerGetAttributes(&attr, kept_idx_host) == cudaSuccess && attr.type == cudaMemoryTypeHost && attr.devicePointer) {
            ctx->kept_mirror = static_cast<int32_t*>(attr.devicePointer);
            mirrored = true;
        } else {
            cudaGetLastError();
        }
    }
    const int erc = keydiff_evict(ctx, k_cache, v_cache, ctx->stage_k[b], ctx->stage_v[b], budget_N, block_B, n_kv_heads,
                                  head_dim, stream);
    ctx->kept_mirror = nullptr;
    if (erc != KEYDIFF_OK) return erc;
    if (capturing == cudaStreamCaptureStatusNone) {
        KD_CUDA(cudaEventRecord(ctx->ev_consumed[b], st));
        ctx->consumed_recorded[b] = true;
    }
    ctx->stage_next = b ^ 1;
    if (kept_idx_host && !mirrored)
        KD_CUDA(cudaMemcpyAsync(kept_idx_host, ctx->kept_idx, sizeof(int32_t) * ctx->U * ctx->cfg.budget,
                                cudaMemcpyDeviceToHost, st));
    if (status_host)
        KD_CUDA(cudaMemcpyAsync(status_host, ctx->status, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    return KEYDIFF_OK;
}

int keydiff_destroy(keydiff_ctx* ctx) {
    if (!ctx) return KEYDIFF_OK;
    int prev = -1;
    cudaGetDevice(&prev);
    cudaSetDevice(ctx->cfg.device);
    cudaDeviceSynchronize();
    free_scratch(ctx);
    if (prev >= 0) cudaSetDevice(prev);
    delete ctx;
    return KEYDIFF_OK;
}

int keydiff_reset(keydiff_ctx* ctx) {
    if (!ctx) return KEYDIFF_ERR_INVALID_ARG;
    ctx->len = 0;
    ctx->anchor_valid = false;
    ctx->next_pos = 0;
    ctx->pos_stale = true;
    return KEYDIFF_OK;
}

int keydiff_set_incremental(keydiff_ctx* ctx, int32_t on) {
    if (!ctx) return KEYDIFF_ERR_INVALID_ARG;
    ctx->incremental = on != 0;
    return KEYDIFF_OK;
}

int keydiff_get_len(const keydiff_ctx* ctx, int32_t* len_out) {
    if (!ctx || !len_out) return KEYDIFF_ERR_INVALID_ARG;
    *len_out = ctx->len;
    return KEYDIFF_OK;
}

int keydiff_set_len(keydiff_ctx* ctx, int32_t len) {
    if (!ctx || len < 0 || len > ctx->cfg.budget) return KEYDIFF_ERR_INVALID_ARG;
    ctx->len = len;
    ctx->anchor_valid = false;   // the caller brought its own cache contents
    ctx->next_pos = len;         // ... which are tokens 0 .. len-1 in token order
    ctx->pos_stale = true;
    return KEYDIFF_OK;
}

int keydiff_get_scratch(const keydiff_ctx* ctx, const float** scores, const int32_t** kept_idx,
                        const int32_t** first_evicted, const int32_t** status) {
    if (!ctx) return KEYDIFF_ERR_INVALID_ARG;
    if (scores) *scores = ctx->scores;
    if (kept_idx) *kept_idx = ctx->kept_idx;
    if (first_evicted) *first_evicted = ctx->first_evicted;
    if (status) *status = ctx->status;
    return KEYDIFF_OK;
}

int keydiff_get_positions(const keydiff_ctx* ctx, const int32_t** pos, long long* next_pos) {
    if (!ctx) return KEYDIFF_ERR_INVALID_ARG;
    if (!slot_reuse(ctx)) return KEYDIFF_ERR_STATE;
    if (pos) *pos = ctx->pos;
    if (next_pos) *next_pos = ctx->next_pos;
    return KEYDIFF_OK;
}

int keydiff_set_positions(keydiff_ctx* ctx, const int32_t* pos_device, int32_t len, long long next_pos, void* stream) {
    if (!ctx || len < 0 || len > ctx->cfg.budget || next_pos < len || next_pos > 0x7fffffffLL) return KEYDIFF_ERR_INVALID_ARG;
    if (!slot_reuse(ctx)) return KEYDIFF_ERR_STATE;
    int dev = -1;
    KD_CUDA(cudaGetDevice(&dev));
    if (dev != ctx->cfg.device) return KEYDIFF_ERR_STATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int total = ctx->U * ctx->cfg.budget;
    if (pos_device) {
        KD_CUDA(cudaMemcpyAsync(ctx->pos, pos_device, sizeof(int32_t) * total, cudaMemcpyDeviceToDevice, st));
    } else {
        kd::pos_iota_kernel<<<(total + 255) / 256, 256, 0, st>>>(ctx->pos, ctx->cfg.budget, total);
        KD_CUDA(cudaGetLastError());
    }
    ctx->len = len;
    ctx->next_pos = next_pos;
    ctx->pos_stale = false;
    ctx->anchor_valid = false;   // the caller brought its own cache contents
    return KEYDIFF_OK;
}

int keydiff_get_moved_rows(const keydiff_ctx* ctx, const unsigned long long** counter) {
    if (!ctx || !counter) return KEYDIFF_ERR_INVALID_ARG;
    *counter = ctx->moved_rows;
    return KEYDIFF_OK;
}

int keydiff_get_launch_info(const keydiff_ctx* ctx, int32_t* path, int32_t* launches_per_step, int32_t* cluster_size) {
    if (!ctx) return KEYDIFF_ERR_INVALID_ARG;
    if (path) *path = ctx->path;
    if (launches_per_step) *launches_per_step = ctx->path == KEYDIFF_PATH_FUSED ? 1 : 4;
    if (cluster_size) *cluster_size = ctx->cluster;
    return KEYDIFF_OK;
}

const char* keydiff_strerror(int code) {
    switch (code) {
        case KEYDIFF_OK: return "ok";
        case KEYDIFF_ERR_INVALID_ARG: return "invalid argument";
        case KEYDIFF_ERR_UNSUPPORTED: return "unsupported configuration or device";
        case KEYDIFF_ERR_ALLOC: return "device memory allocation failed";
        case KEYDIFF_ERR_CUDA: return "CUDA runtime error";
        case KEYDIFF_ERR_STATE: return "call not valid in the current state (is the ctx's device current?)";
        case KEYDIFF_ERR_TIMEOUT: return "bounded device-side wait expired";
        case KEYDIFF_ERR_TOO_LARGE: return "request needs more scratch than the built-in static scratch array holds";
        case KEYDIFF_ERR_INTERNAL: return "a kernel computed a row index outside its tensor (debug-checks build)";
        default: return "unknown keydiff status";
    }
}

int keydiff_last_cuda_error(void) { return g_last_cuda_error; }

int keydiff_selftest_bounded_wait(int32_t* status_device, int32_t polls, void* stream) {
    if (!status_device || polls < 1 || polls > 4096) return KEYDIFF_ERR_INVALID_ARG;
    kd::bounded_wait_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(status_device, static_cast<uint32_t>(polls));
    KD_CUDA(cudaGetLastError());
    return KEYDIFF_OK;
}

#ifdef KEYDIFF_PHASE_STAMPS
// Phase-stamp build only: copies the per-CTA, per-phase nanosecond totals of the fused kernel to out_host
// ([ctas][16] unsigned 64-bit, ctas <= 2368) and optionally clears them.  Synchronises the device.
__attribute__((visibility("default"))) int keydiff_debug_phase_ns(unsigned long long* out_host, int32_t ctas, int32_t reset) {
    if (!out_host || ctas < 1 || ctas > kd::kMaxStampCtas) return KEYDIFF_ERR_INVALID_ARG;
    KD_CUDA(cudaDeviceSynchronize());
    KD_CUDA(cudaMemcpyFromSymbol(out_host, kd::g_phase_ns, sizeof(unsigned long long) * ctas * kd::kMaxPhases));
    if (reset) {
        void* addr = nullptr;
        KD_CUDA(cudaGetSymbolAddress(&addr, kd::g_phase_ns));
        KD_CUDA(cudaMemset(addr, 0, sizeof(unsigned long long) * kd::kMaxStampCtas * kd::kMaxPhases));
    }
    return KEYDIFF_OK;
}
#endif

int keydiff_debug_fail_alloc(int32_t nth) {
    if (nth < 0) return KEYDIFF_ERR_INVALID_ARG;
    g_fail_alloc_countdown = nth;
    return KEYDIFF_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Allocation-free entry point.
//
// Some callers cannot allocate device memory at all: code running inside a serving process whose
// memory pool already owns the whole GPU (any cudaMalloc would fail or fragment the pool), plugin
// code that is only handed tensors, and set-ups where allocation is forbidden after start-up
// because it synchronises the device.  keydiff_create needs cudaMalloc for its scratch, so such
// callers get keydiff_evict_static instead: the same staged kernels, with their scratch carved
// out of one array that is part of the library image.
//
// The array's name below is, in host code, only a handle for the runtime -- it is NOT a device
// address, and a kernel handed it directly would read the wrong memory.  The device address is
// looked up once per device with cudaGetSymbolAddress (with that device current) and cached.
namespace {

constexpr size_t kStaticScratchBytes = 16u << 20;   // 16 MiB, resident on every GPU that loads the library
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxStaticDevices = 64;
unsigned char* g_static_scratch_addr[kMaxStaticDevices] = {};   // device address per device ordinal
std::mutex g_static_mutex;

// Resolve (once per device) the device address of the scratch array for the CURRENT device and
// raise the select kernel's dynamic shared-memory limit there.
int static_scratch_for_current_device(unsigned char** out) {
    int dev = -1;
    KD_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxStaticDevices) return KEYDIFF_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_scratch_addr[dev]) {
        int major = 0;
        KD_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
        if (major != 10) return KEYDIFF_ERR_UNSUPPORTED;
        void* addr = nullptr;
        KD_CUDA(cudaGetSymbolAddress(&addr, g_static_scratch));
        KD_CUDA(cudaFuncSetAttribute(kd::select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSelectSmem));
        g_static_scratch_addr[dev] = static_cast<unsigned char*>(addr);
    }
    *out = g_static_scratch_addr[dev];
    return KEYDIFF_OK;
}

inline size_t round256(size_t b) { return (b + 255) & ~static_cast<size_t>(255); }

}  // namespace

extern "C" int keydiff_evict_static(void* k_cache, void* v_cache, const void* new_k, const void* new_v,
                                    int32_t len, int32_t budget_N, int32_t block_B, int32_t n_units,
                                    int32_t head_dim, float eps, void* stream) {
    using namespace kd;
    if (!k_cache || !v_cache || !new_k || !new_v) return KEYDIFF_ERR_INVALID_ARG;
    if (!aligned16(k_cache) || !aligned16(v_cache) || !aligned16(new_k) || !aligned16(new_v)) return KEYDIFF_ERR_INVALID_ARG;
    if (k_cache == v_cache || k_cache == new_k || v_cache == new_v) return KEYDIFF_ERR_INVALID_ARG;
    if (budget_N < 1 || block_B < 1 || n_units < 1 || len < 0 || len > budget_N || eps < 0.f) return KEYDIFF_ERR_INVALID_ARG;
    if (head_dim != kHeadDim) return KEYDIFF_ERR_UNSUPPORTED;
    if (n_units > 65535) return KEYDIFF_ERR_TOO_LARGE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint4* kc = static_cast<uint4*>(k_cache);
    uint4* vc = static_cast<uint4*>(v_cache);
    const uint4* nk = static_cast<const uint4*>(new_k);
    const uint4* nv = static_cast<const uint4*>(new_v);
    const long long n = static_cast<long long>(len) + block_B;
    const int N = budget_N, U = n_units;
    // set-up (first call on a device only) comes before anything is enqueued, whatever kind of step this is
    unsigned char* base = nullptr;
    const int src = static_scratch_for_current_device(&base);
    if (src != KEYDIFF_OK) return src;
    {
        // the tensors must live on the current device: the scratch address was looked up for it
        int dev = -1;
        KD_CUDA(cudaGetDevice(&dev));
        cudaPointerAttributes attr;
        if (cudaPointerGetAttributes(&attr, k_cache) != cudaSuccess) { cudaGetLastError(); return KEYDIFF_ERR_INVALID_ARG; }
        if (attr.type == cudaMemoryTypeDevice && attr.device != dev) return KEYDIFF_ERR_STATE;
    }
    if (n <= N) {   // budget not exceeded: plain append, no scratch involved
        const int threads = 256;
        const dim3 grid((block_B * kRowVec + threads - 1) / threads, U, 2);
        append_kernel<<<grid, threads, 0, st>>>(kc, vc, nk, nv, len, block_B, N);
        KD_CUDA(cudaGetLastError());
        return KEYDIFF_OK;
    }
    if (n * 4 > kMaxSelectSmem) return KEYDIFF_ERR_TOO_LARGE;
    const int splits = static_cast<int>(std::max(1LL, std::min({(592LL + U - 1) / U, (n + 63) / 64, 64LL})));
    // carve the static array: [moved counter][partials][norms][scores][kept_idx][first_evicted]
    size_t off = 0;
    auto take = [&off](size_t bytes) { const size_t o = off; off += round256(bytes); return o; };
    const size_t o_moved = take(sizeof(unsigned long long));
    const size_t o_partial = take(sizeof(double) * U * splits * kHeadDim);
    const size_t o_norms = take(sizeof(float) * U * n);
    const size_t o_scores = take(sizeof(float) * U * n);
    const size_t o_kept = take(sizeof(int32_t) * static_cast<size_t>(U) * N);
    const size_t o_first = take(sizeof(int32_t) * U);
    if (off > kStaticScratchBytes) return KEYDIFF_ERR_TOO_LARGE;
    unsigned long long* moved = reinterpret_cast<unsigned long long*>(base + o_moved);
    double* partial = reinterpret_cast<double*>(base + o_partial);
    float* norms = reinterpret_cast<float*>(base + o_norms);
    float* scores = reinterpret_cast<float*>(base + o_scores);
    int32_t* kept = reinterpret_cast<int32_t*>(base + o_kept);
    int32_t* first = reinterpret_cast<int32_t*>(base + o_first);
    // the array still holds the previous call's contents; the counter accumulates, so it is the
    // one part that must start from zero (everything else is fully overwritten before it is read)
    KD_CUDA(cudaMemsetAsync(moved, 0, sizeof(unsigned long long), st));
    const float e = eps > 0.f ? eps : kDefaultEps;
    const int nn = static_cast<int>(n);
    const int rows_per_split = (nn + splits - 1) / splits;
    const dim3 grid(splits, U);
    anchor_partial_kernel<<<grid, kStagedThreads, 0, st>>>(kc, nk, len, block_B, N, e, rows_per_split, nn, partial, norms, 0);
    score_kernel<<<grid, kStagedThreads, 0, st>>>(kc, nk, len, block_B, N, e, rows_per_split, nn, partial, norms, scores);
    select_kernel<<<U, kSelectThreads, static_cast<size_t>(nn) * 4, st>>>(scores, nn, N, nn, len, kept, first, moved, 0, nullptr, 0);
    compact_kernel<<<dim3(2, U), kCompactThreads, 0, st>>>(kc, vc, nk, nv, len, block_B, N, kept, first, nullptr);
    KD_CUDA(cudaGetLastError());
    return KEYDIFF_OK;
}
