// Fused path: ONE launch per evicting step.  A thread-block cluster of C CTAs owns one unit
// (one KV head of one layer of one sequence) from the anchor to the compacted K and V:
//
//   load K      every CTA pulls its contiguous slice of the unit's n key rows on chip exactly
//               once: most rows into shared memory with TMA bulk copies (cp.async.bulk +
//               mbarrier, all chunks in flight at once), the remainder into registers with
//               128-bit loads.  Nothing is read from HBM twice.
//   a1 anchor   per-row norm, sum of k/||k|| per CTA, partial sums combined across the cluster
//               through distributed shared memory in a fixed order (App. B.1, expr. 1).
//   a2 scores   e_i = -(mu.k_i)/max(||mu|| ||k_i||, eps) from the on-chip rows; the fp32 score goes
//               to global scratch and its orderable key is pushed into every CTA's key table
//               through DSMEM (App. B.1, expr. 2).
//   a3 select   every CTA finds the N-th largest key of the full table locally: a 2048-bin
//               histogram over the (monotone) fixed-point image of e, then an exact rank among
//               the few keys of the threshold bin; a 4x8-bit radix select is the fallback when
//               that bin is crowded.  Ties keep the older token (Eq. efficient-keydiff, topk).
//   a4 compact  an ordered scan gives every kept row its destination; K rows are written from
//               chip to their new place, then the slice's V rows take the same trip (load all,
//               cluster barrier, store all) -- in place, original token order (Eq. keydiff).
//
// In-place safety: every source row of the unit is on chip (in some CTA of the cluster)
// before the first destination row is written -- for K by the barrier after the score pass, for
// V by an explicit cluster barrier between its loads and its stores -- so no store can
// overwrite a row that is still to be read.
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
constexpr int kChunkRows = kGroups;                     // one bulk-load chunk = one row per group
constexpr int kMaxChunks = 13;                          // <= 832 rows of a slice live in shared memory
constexpr int kRegRows = 6;                             // + up to 6 rows per group (384 rows) in registers
constexpr int kBins = 2048;                             // first-level histogram over e in [-1, 1]
constexpr int kCandCap = kFusedThreads;                 // exact-rank stage handles this many candidates
constexpr int kSmemLimit = 232448;                      // opt-in shared memory per CTA on sm_100
constexpr int kErrTimeout = -6;                         // KEYDIFF_ERR_TIMEOUT
constexpr uint32_t kWaitSpins = 1u << 24;               // bound of every mbarrier wait

struct FusedLayout {
    int rows, keys, work, cand_key, cand_idx, norms, sel, partial, mu, mbar, misc, total;
};

// Shared-memory carve-up for a slice with `smem_rows` resident rows and a key table of nkeys.
__host__ __device__ inline FusedLayout fused_layout(int smem_rows, int nkeys) {
    FusedLayout L;
    int off = 0;
    auto take = [&off](int bytes) { const int o = off; off += (bytes + 127) & ~127; return o; };
    L.rows = take(smem_rows * kRowBytes);
    L.keys = take(nkeys * 4);
    L.work = take(kBins * 4);   // histogram / warp-reduction scratch / destination table (never live together)
    L.cand_key = take(kCandCap * 4);
    L.cand_idx = take(kCandCap * 4);
    L.norms = take(smem_rows * 4);
    L.sel = take(static_cast<int>(sizeof(SelectSmem)));
    L.partial = take(kHeadDim * 4);
    L.mu = take(kHeadDim * 4);
    L.mbar = take(kMaxChunks * 8);
    L.misc = take(64);
    L.total = off;
    return L;
}

struct FusedParams {
    uint4* k_cache; uint4* v_cache; const uint4* new_k; const uint4* new_v;
    int len, B, N, U;
    float eps;
    int cluster;        // CTAs per cluster
    int rows_per_cta;   // slice length = ceil(n / cluster)
    int smem_rows;      // rows of a slice held in shared memory (multiple of kChunkRows)
    int nkeys;          // key-table capacity (>= n)
    int nmax;           // row stride of the score scratch
    float* scores; int32_t* kept_idx; int32_t* first_evicted;
    unsigned long long* moved_rows; int32_t* status;
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ uint32_t cluster_ctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r; asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank)); return r;
}
__device__ __forceinline__ float ld_cluster_f32(uint32_t addr) {
    float v; asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory"); return v;
}
__device__ __forceinline__ void st_cluster_u32(uint32_t addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
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
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Bounded wait; returns false (and records the timeout) if the phase never completed.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int32_t* status) {
    for (uint32_t spin = 0; spin < kWaitSpins; ++spin)
        if (mbar_try_wait(bar, parity)) return true;
    atomicExch(status, kErrTimeout);
    return false;
}

// fixed-point image of an orderable key: monotone non-decreasing in e, 2048 bins over [-1, 1]
__device__ __forceinline__ int key_bin(uint32_t key) {
    const uint32_t u = (key & 0x80000000u) ? (key & 0x7fffffffu) : ~key;   // inverse of order_key
    const int q = __float2int_rd((__uint_as_float(u) + 1.0f) * 1024.0f);
    return min(max(q, 0), kBins - 1);
}

// Thread 0: start the bulk loads of this CTA's resident rows [0, rs) of a slice starting at unit
// row seg_a, one mbarrier per chunk of 64 rows; chunks that end at or before skip_local are left
// out.  Rows below `len` come from the cache tensor, the rest from the block tensor.
__device__ __forceinline__ void issue_slice_loads(const uint4* cache, const uint4* block, int u, int len, int B, int N,
                                                  int seg_a, int rs, int skip_local, uint32_t rows_sa, uint32_t mbar_sa) {
    for (int j = 0; j * kChunkRows < rs; ++j) {
        const int lo = j * kChunkRows, hi = min(rs, lo + kChunkRows);
        if (hi <= skip_local) continue;
        const int g0 = seg_a + lo;                               // first unit row of the chunk
        const int from_cache = min(max(len - g0, 0), hi - lo);
        const int from_block = (hi - lo) - from_cache;
        const uint32_t bar = mbar_sa + 8 * j, dst = rows_sa + lo * kRowBytes;
        mbar_expect_tx(bar, (hi - lo) * kRowBytes);
        if (from_cache > 0)
            bulk_load(dst, cache + (static_cast<size_t>(u) * N + g0) * kRowVec, from_cache * kRowBytes, bar);
        if (from_block > 0)
            bulk_load(dst + from_cache * kRowBytes,
                      block + (static_cast<size_t>(u) * B + (g0 + from_cache - len)) * kRowVec, from_block * kRowBytes, bar);
    }
}

__global__ void __launch_bounds__(kFusedThreads, 1) fused_evict_kernel(const FusedParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    const FusedLayout L = fused_layout(p.smem_rows, p.nkeys);
    uint4* rows = reinterpret_cast<uint4*>(smem + L.rows);
    uint32_t* keys = reinterpret_cast<uint32_t*>(smem + L.keys);
    int* hist = reinterpret_cast<int*>(smem + L.work);
    float* red = reinterpret_cast<float*>(smem + L.work);
    int* dst_of = reinterpret_cast<int*>(smem + L.work);
    uint32_t* cand_key = reinterpret_cast<uint32_t*>(smem + L.cand_key);
    int* cand_idx = reinterpret_cast<int*>(smem + L.cand_idx);
    float* norms = reinterpret_cast<float*>(smem + L.norms);
    SelectSmem& sel = *reinterpret_cast<SelectSmem*>(smem + L.sel);
    float* partial = reinterpret_cast<float*>(smem + L.partial);
    float* mu_sh = reinterpret_cast<float*>(smem + L.mu);
    int* misc = reinterpret_cast<int*>(smem + L.misc);   // 0 ncand, 1 first_evicted, 2 need_eq, 3 T, 4 winner idx, 5 m (float)
    const uint32_t rows_sa = smem_addr(rows), mbar_sa = smem_addr(smem + L.mbar);
    const uint32_t keys_sa = smem_addr(keys), partial_sa = smem_addr(partial);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = tid >> 3, t = tid & 7;
    const int C = p.cluster;
    const int crank = static_cast<int>(cluster_ctarank());
    const int cluster_id = blockIdx.x / C, nclusters = gridDim.x / C;
    const int len = p.len, B = p.B, N = p.N, n = len + B;
    const int seg_a = min(n, crank * p.rows_per_cta), seg_b = min(n, seg_a + p.rows_per_cta), seg = seg_b - seg_a;
    const int rs = min(seg, p.smem_rows);            // slice rows resident in shared memory
    const int nchunks = (rs + kChunkRows - 1) / kChunkRows;

    if (tid == 0) {
        for (int j = 0; j < kMaxChunks; ++j) mbar_init(mbar_sa + 8 * j, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    uint32_t parity = 0;   // bit j: phase parity the next wait on chunk j's mbarrier expects

    for (int u = cluster_id; u < p.U; u += nclusters) {
        // ------------------------------------------------------------ load K (once)
        if (tid == 0) {
            fence_proxy_async();
            issue_slice_loads(p.k_cache, p.new_k, u, len, B, N, seg_a, rs, -1, rows_sa, mbar_sa);
        }
        uint4 ra[kRegRows], rb[kRegRows];   // register-resident rows: local row rs + 64k + g
        float rn[kRegRows];
#pragma unroll
        for (int k = 0; k < kRegRows; ++k) {
            const int lr = rs + k * kGroups + g;
            ra[k] = make_uint4(0, 0, 0, 0); rb[k] = ra[k];
            if (lr < seg) {
                const uint4* row = concat_row(p.k_cache, p.new_k, u, seg_a + lr, len, B, N);
                ra[k] = row[t]; rb[k] = row[t + 8];
            }
        }
        // ------------------------------------------------------------ a1: norms and anchor partial
        float acc[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) acc[j] = 0.f;
        for (int j = 0; j < nchunks; ++j) {
            mbar_wait(mbar_sa + 8 * j, (parity >> j) & 1u, p.status);
            const int lr = j * kChunkRows + g;
            const bool valid = lr < rs;
            uint4 a = make_uint4(0, 0, 0, 0), b = a;
            if (valid) { a = rows[lr * kRowVec + t]; b = rows[lr * kRowVec + t + 8]; }
            float x[16];
            unpack_row(a, b, x);
            const float r = sqrtf(row_sumsq(x));
            const float inv = 1.0f / fmaxf(r, p.eps);
            if (valid) {
#pragma unroll
                for (int q = 0; q < 16; ++q) acc[q] = fmaf(x[q], inv, acc[q]);
                if (t == 0) norms[lr] = r;
            }
        }
        parity ^= (1u << nchunks) - 1u;
#pragma unroll
        for (int k = 0; k < kRegRows; ++k) {
            float x[16];
            unpack_row(ra[k], rb[k], x);
            const float r = sqrtf(row_sumsq(x));
            const float inv = 1.0f / fmaxf(r, p.eps);
            rn[k] = r;
            if (rs + k * kGroups + g < seg) {
#pragma unroll
                for (int q = 0; q < 16; ++q) acc[q] = fmaf(x[q], inv, acc[q]);
            }
        }
        // CTA reduction: 4 groups of a warp by shuffle, 16 warps through shared memory, fixed order
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            float v = acc[q];
            v += __shfl_xor_sync(0xffffffffu, v, 8);
            v += __shfl_xor_sync(0xffffffffu, v, 16);
            acc[q] = v;
        }
        if (lane < 8) {
#pragma unroll
            for (int q = 0; q < 16; ++q) red[warp * kHeadDim + lane_channel(t, q)] = acc[q];
        }
        __syncthreads();
        if (tid < kHeadDim) {
            float s = 0.f;
            for (int w = 0; w < kFusedWarps; ++w) s += red[w * kHeadDim + tid];
            partial[tid] = s;
        }
        cluster_sync_all();   // (1) every CTA's partial is written; all K rows of the unit are on chip
        if (tid < kHeadDim) {
            float s = 0.f;
            for (int c = 0; c < C; ++c) s += ld_cluster_f32(map_to_cta(partial_sa + 4 * tid, c));   // fixed order
            mu_sh[tid] = s / static_cast<float>(n);
        }
        __syncthreads();
        if (warp == 0) {
            float v = 0.f;
#pragma unroll
            for (int q = 0; q < 4; ++q) { const float w = mu_sh[lane * 4 + q]; v = fmaf(w, w, v); }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == 0) reinterpret_cast<float*>(misc)[5] = sqrtf(v);
        }
        __syncthreads();
        // ------------------------------------------------------------ a2: scores, keys pushed to every CTA
        {
            float w[16];
#pragma unroll
            for (int q = 0; q < 16; ++q) w[q] = mu_sh[lane_channel(t, q)];
            const float m = reinterpret_cast<float*>(misc)[5];
            for (int j = 0; j < nchunks; ++j) {
                const int lr = j * kChunkRows + g;
                const bool valid = lr < rs;
                uint4 a = make_uint4(0, 0, 0, 0), b = a;
                if (valid) { a = rows[lr * kRowVec + t]; b = rows[lr * kRowVec + t + 8]; }
                float x[16];
                unpack_row(a, b, x);
                const float dot = row_dot(x, w);
                if (valid) {
                    const float e = eviction_score(dot, m, norms[lr], p.eps);
                    const int i = seg_a + lr;
                    if (t == 0) p.scores[static_cast<size_t>(u) * p.nmax + i] = e;
                    const uint32_t key = order_key(e);
                    for (int c = t; c < C; c += kLanesPerRow) st_cluster_u32(map_to_cta(keys_sa + 4 * i, c), key);
                }
            }
#pragma unroll
            for (int k = 0; k < kRegRows; ++k) {
                float x[16];
                unpack_row(ra[k], rb[k], x);
                const float dot = row_dot(x, w);
                const int lr = rs + k * kGroups + g;
                if (lr < seg) {
                    const float e = eviction_score(dot, m, rn[k], p.eps);
                    const int i = seg_a + lr;
                    if (t == 0) p.scores[static_cast<size_t>(u) * p.nmax + i] = e;
                    const uint32_t key = order_key(e);
                    for (int c = t; c < C; c += kLanesPerRow) st_cluster_u32(map_to_cta(keys_sa + 4 * i, c), key);
                }
            }
        }
        cluster_sync_all();   // (2) the key table of every CTA holds all n keys
        // ------------------------------------------------------------ a3: N-th largest key
        for (int b = tid; b < kBins; b += kFusedThreads) hist[b] = 0;
        if (tid == 0) { misc[0] = 0; misc[1] = n; misc[2] = 0; }
        __syncthreads();
        for (int i = tid; i < n; i += kFusedThreads) atomicAdd(&hist[key_bin(keys[i])], 1);
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
        for (int i = tid; i < n; i += kFusedThreads) {
            const uint32_t k = keys[i];
            if (key_bin(k) == bstar) {
                const int slot = atomicAdd(&misc[0], 1);
                if (slot < kCandCap) { cand_key[slot] = k; cand_idx[slot] = i; }
            }
        }
        __syncthreads();
        Threshold th;
        const int ncand = misc[0];
        if (ncand <= kCandCap) {
            // exact rank among the candidates under (key desc, index asc)
            if (tid < ncand) {
                const uint32_t mk = cand_key[tid];
                const int mi = cand_idx[tid];
                int rank = 0;
                for (int q = 0; q < ncand; ++q) {
                    const uint32_t ok = cand_key[q];
                    rank += (ok > mk) || (ok == mk && cand_idx[q] < mi);
                }
                if (rank == need - 1) { misc[3] = static_cast<int>(mk); misc[4] = mi; }
            }
            __syncthreads();
            if (tid < ncand && cand_key[tid] == static_cast<uint32_t>(misc[3]) && cand_idx[tid] <= misc[4])
                atomicAdd(&misc[2], 1);
            __syncthreads();
            th.key = static_cast<uint32_t>(misc[3]);
            th.need_eq = misc[2];
        } else {
            th = block_radix_select<kFusedThreads>(keys, n, N, sel);
        }
        // ------------------------------------------------------------ plan: destination of every kept row
        {
            const int per = (n + kFusedThreads - 1) / kFusedThreads;
            const int i0 = min(n, tid * per), i1 = min(n, i0 + per);
            int gt = 0, eq = 0;
            for (int i = i0; i < i1; ++i) { const uint32_t k = keys[i]; gt += k > th.key; eq += k == th.key; }
            int pre_gt, pre_eq, tot_gt, tot_eq;
            block_exclusive_scan2<kFusedThreads>(gt, eq, sel, pre_gt, pre_eq, tot_gt, tot_eq);
            int local_first = n;
            for (int i = i0; i < i1; ++i) {
                const uint32_t k = keys[i];
                const bool is_eq = k == th.key;
                const bool keep = k > th.key || (is_eq && pre_eq < th.need_eq);
                if (i >= seg_a && i < seg_b) dst_of[i - seg_a] = keep ? pre_gt + min(pre_eq, th.need_eq) : -1;
                if (!keep) local_first = min(local_first, i);
                pre_gt += k > th.key;
                pre_eq += is_eq;
            }
            if (local_first < n) atomicMin(&misc[1], local_first);
            __syncthreads();
        }
        const int first_evicted = misc[1];
        const int first_moved = min(first_evicted, len);   // block rows always move into the cache
        if (crank == 0 && tid == 0) {
            p.first_evicted[u] = first_evicted;
            atomicAdd(p.moved_rows, static_cast<unsigned long long>(N - first_moved));
        }
        for (int lr = tid; lr < seg; lr += kFusedThreads) {
            const int d = dst_of[lr];
            if (d >= 0) p.kept_idx[static_cast<size_t>(u) * N + d] = seg_a + lr;
        }
        // ------------------------------------------------------------ a4: K rows to their new place
        {
            uint4* out = p.k_cache + static_cast<size_t>(u) * N * kRowVec;
            for (int q = tid; q < rs * kRowVec; q += kFusedThreads) {
                const int lr = q >> 4, d = dst_of[lr];
                if (d >= 0 && seg_a + lr >= first_moved) out[d * kRowVec + (q & 15)] = rows[q];
            }
#pragma unroll
            for (int k = 0; k < kRegRows; ++k) {
                const int lr = rs + k * kGroups + g;
                if (lr < seg) {
                    const int d = dst_of[lr];
                    if (d >= 0 && seg_a + lr >= first_moved) { out[d * kRowVec + t] = ra[k]; out[d * kRowVec + t + 8] = rb[k]; }
                }
            }
        }
        __syncthreads();   // shared-memory rows are free again
        // ------------------------------------------------------------ a4: V rows: load all, barrier, store all
        const int skip_local = first_moved - seg_a;   // local rows below this did not move
        if (tid == 0) {
            fence_proxy_async();
            issue_slice_loads(p.v_cache, p.new_v, u, len, B, N, seg_a, rs, skip_local, rows_sa, mbar_sa);
        }
#pragma unroll
        for (int k = 0; k < kRegRows; ++k) {
            const int lr = rs + k * kGroups + g;
            if (lr < seg && lr >= skip_local) {
                const uint4* row = concat_row(p.v_cache, p.new_v, u, seg_a + lr, len, B, N);
                ra[k] = row[t]; rb[k] = row[t + 8];
            }
        }
        for (int j = 0; j < nchunks; ++j) {
            if (min(rs, (j + 1) * kChunkRows) <= skip_local) continue;   // chunk was not loaded
            mbar_wait(mbar_sa + 8 * j, (parity >> j) & 1u, p.status);
            parity ^= 1u << j;
        }
        cluster_sync_all();   // (3) every V row of the unit that moves is on chip
        {
            uint4* out = p.v_cache + static_cast<size_t>(u) * N * kRowVec;
            for (int q = tid; q < rs * kRowVec; q += kFusedThreads) {
                const int lr = q >> 4, d = dst_of[lr];
                if (d >= 0 && lr >= skip_local) out[d * kRowVec + (q & 15)] = rows[q];
            }
#pragma unroll
            for (int k = 0; k < kRegRows; ++k) {
                const int lr = rs + k * kGroups + g;
                if (lr < seg && lr >= skip_local) {
                    const int d = dst_of[lr];
                    if (d >= 0) { out[d * kRowVec + t] = ra[k]; out[d * kRowVec + t + 8] = rb[k]; }
                }
            }
        }
        __syncthreads();   // rows / dst_of are free for the next unit
    }
    cluster_sync_all();   // no CTA leaves while a peer may still address its shared memory
}

}  // namespace kd
