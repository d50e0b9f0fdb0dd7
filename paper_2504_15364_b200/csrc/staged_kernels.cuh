// Staged path: four launches per evicting step (anchor partials -> scores -> select ->
// compaction) plus the append copy.  Serves any unit size whose score vector fits one CTA's
// shared memory; the fused cluster kernel is preferred when a unit's keys fit a cluster.
#pragma once
#include "common.cuh"
#include "select.cuh"

namespace kd {

constexpr int kStagedThreads = 256;          // anchor / score kernels: 32 row groups per CTA
constexpr int kSelectThreads = 1024;
constexpr int kCompactThreads = 512;
constexpr int kCompactRows = 128;            // rows staged per iteration (32 KB)

// Row i of the logical concatenation [K_cache || k_block] of unit u (Eq. block_processing).
__device__ __forceinline__ const uint4* concat_row(const uint4* cache, const uint4* block,
                                                   int u, int i, int len, int B, int N) {
    return i < len ? cache + (static_cast<size_t>(u) * N + i) * kRowVec
                   : block + (static_cast<size_t>(u) * B + (i - len)) * kRowVec;
}

// Step a1 (App. B.1, first expression): per key ||k_i|| and the partial sum of k_i/max(||k_i||,eps)
// (of k_i itself for the raw-mean anchor of Sec. 3.2) over this CTA's slice of rows.  grid = (splits, U).
__global__ void __launch_bounds__(kStagedThreads)
anchor_partial_kernel(const uint4* __restrict__ k_cache, const uint4* __restrict__ new_k,
                      int len, int B, int N, float eps, int rows_per_split, int nmax,
                      double* __restrict__ partial, float* __restrict__ norms, int raw_anchor) {
    __shared__ double red[kStagedThreads / kLanesPerRow][kHeadDim + 2];
    const int u = blockIdx.y, s = blockIdx.x, splits = gridDim.x;
    const int n = len + B;
    const int r0 = s * rows_per_split, r1 = min(n, r0 + rows_per_split);
    const int g = threadIdx.x >> 3, t = threadIdx.x & 7;
    // a thread adds four rows in fp32, then carries the sums on in double: the anchor is a sum of thousands of
    // unit vectors that cancels when the keys point in many directions
    double wide[16];
    float acc[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) { wide[j] = 0.0; acc[j] = 0.f; }
    int pending = 0;
    for (int base = r0; base < r1; base += kStagedThreads / kLanesPerRow) {
        const int i = base + g;
        const bool valid = i < r1;
        uint4 a = make_uint4(0, 0, 0, 0), b = a;
        if (valid) {
            const uint4* row = concat_row(k_cache, new_k, u, i, len, B, N);
            a = row[t]; b = row[t + 8];
        }
        float x[16];
        unpack_row(a, b, x);
        const float r = sqrtf(row_sumsq(x));
        const float inv = raw_anchor ? 1.0f : 1.0f / fmaxf(r, eps);   // raw-mean anchor: the keys themselves are summed
        if (valid) {
#pragma unroll
            for (int j = 0; j < 16; ++j) acc[j] = fmaf(x[j], inv, acc[j]);
            if (t == 0) norms[static_cast<size_t>(u) * nmax + i] = r;
        }
        if (++pending == 4) {
#pragma unroll
            for (int j = 0; j < 16; ++j) { wide[j] += static_cast<double>(acc[j]); acc[j] = 0.f; }
            pending = 0;
        }
    }
#pragma unroll
    for (int j = 0; j < 16; ++j) red[g][lane_channel(t, j)] = wide[j] + static_cast<double>(acc[j]);
    __syncthreads();
    if (threadIdx.x < kHeadDim) {
        double sum = 0.0;
        for (int q = 0; q < kStagedThreads / kLanesPerRow; ++q) sum += red[q][threadIdx.x];   // fixed order
        partial[(static_cast<size_t>(u) * splits + s) * kHeadDim + threadIdx.x] = sum;
    }
}

// Step a2 (App. B.1, second expression): anchor = (sum of partials)/n, its norm, then
// e_i = -(mu.k_i)/max(||mu||*||k_i||, eps) for this CTA's slice.  grid = (splits, U).
__global__ void __launch_bounds__(kStagedThreads)
score_kernel(const uint4* __restrict__ k_cache, const uint4* __restrict__ new_k,
             int len, int B, int N, float eps, int rows_per_split, int nmax,
             const double* __restrict__ partial, const float* __restrict__ norms,
             float* __restrict__ scores) {
    __shared__ float mu_sh[kHeadDim];
    __shared__ float m_sh;
    const int u = blockIdx.y, s = blockIdx.x, splits = gridDim.x;
    const int n = len + B;
    if (threadIdx.x < kHeadDim) {
        double sum = 0.0;
        for (int q = 0; q < splits; ++q) sum += partial[(static_cast<size_t>(u) * splits + q) * kHeadDim + threadIdx.x];
        mu_sh[threadIdx.x] = static_cast<float>(sum / static_cast<double>(n));
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        float v = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) { const float w = mu_sh[threadIdx.x * 4 + j]; v = fmaf(w, w, v); }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (threadIdx.x == 0) m_sh = sqrtf(v);
    }
    __syncthreads();
    const int g = threadIdx.x >> 3, t = threadIdx.x & 7;
    float w[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) w[j] = mu_sh[lane_channel(t, j)];
    const float m = m_sh;
    const int r0 = s * rows_per_split, r1 = min(n, r0 + rows_per_split);
    for (int base = r0; base < r1; base += kStagedThreads / kLanesPerRow) {
        const int i = base + g;
        const bool valid = i < r1;
        uint4 a = make_uint4(0, 0, 0, 0), b = a;
        if (valid) {
            const uint4* row = concat_row(k_cache, new_k, u, i, len, B, N);
            a = row[t]; b = row[t + 8];
        }
        float x[16];
        unpack_row(a, b, x);
        const float dot = row_dot(x, w);
        if (valid && t == 0) {
            const float r = norms[static_cast<size_t>(u) * nmax + i];
            scores[static_cast<size_t>(u) * nmax + i] = eviction_score(dot, m, r, eps);
        }
    }
}

// Step a3 + the plan for a4: exact N-th largest eviction score (ties by index), then the
// ascending list of kept token indices.  grid = U, dynamic smem = n * 4 bytes.
__global__ void __launch_bounds__(kSelectThreads)
select_kernel(const float* __restrict__ scores, int n, int N, int nmax, int len,
              int32_t* __restrict__ kept_idx, int32_t* __restrict__ first_evicted,
              unsigned long long* __restrict__ moved_rows, int window,
              const int32_t* __restrict__ pos, int next_pos) {
    extern __shared__ uint32_t keys[];
    __shared__ SelectSmem sm;
    const int u = blockIdx.x, tid = threadIdx.x;
    // sliding window (Sec. 3.2): the last `window` tokens carry the largest possible key, so the top-N
    // selection keeps them all and fills the other N - window places by score.  With slot reuse (pos !=
    // nullptr) the cache is not in token order and "last" is read off the slots' token positions.
    const int first_recent = next_pos + (n - len) - window;
    for (int i = tid; i < n; i += kSelectThreads) {
        const bool recent = pos ? (i < len ? pos[static_cast<size_t>(u) * N + i] : next_pos + (i - len)) >= first_recent
                                : i >= n - window;
        keys[i] = recent ? 0xffffffffu : order_key(scores[static_cast<size_t>(u) * nmax + i]);
    }
    if (tid == 0) sm.first_evicted = n;
    __syncthreads();
    const Threshold th = block_radix_select<kSelectThreads>(keys, n, N, sm);
    // each thread owns a contiguous run of tokens so that prefixes follow token order
    const int per = (n + kSelectThreads - 1) / kSelectThreads;
    const int i0 = min(n, tid * per), i1 = min(n, i0 + per);
    int gt = 0, eq = 0;
    for (int i = i0; i < i1; ++i) { const uint32_t k = keys[i]; gt += k > th.key; eq += k == th.key; }
    int pre_gt, pre_eq, tot_gt, tot_eq;
    block_exclusive_scan2<kSelectThreads>(gt, eq, sm, pre_gt, pre_eq, tot_gt, tot_eq);
    int local_first = n;
    for (int i = i0; i < i1; ++i) {
        const uint32_t k = keys[i];
        const bool is_eq = k == th.key;
        const bool keep = k > th.key || (is_eq && pre_eq < th.need_eq);
        if (keep) kept_idx[static_cast<size_t>(u) * N + pre_gt + min(pre_eq, th.need_eq)] = i;
        else local_first = min(local_first, i);
        pre_gt += k > th.key;
        pre_eq += is_eq;
    }
    if (local_first < n) atomicMin(&sm.first_evicted, local_first);
    __syncthreads();
    if (tid == 0) {
        first_evicted[u] = sm.first_evicted;
        // block rows always move into the cache, cache rows only from the first evicted one on
        // (with slot reuse the placement kernel counts the rows it writes)
        if (!pos) atomicAdd(moved_rows, static_cast<unsigned long long>(N - min(len, sm.first_evicted)));
    }
}

// Step a4: K' = gather(K,S), V' = gather(V,S) in token order, in place.  One CTA per
// (tensor, unit) walks the destination rows left to right in chunks: a chunk's source rows are
// all read into shared memory before any of its destination rows is written, and because every
// source index is >= its destination index, later chunks never need a row an earlier chunk
// overwrote.  Rows in front of the first evicted row stay where they are.  grid = (2, U).
__global__ void __launch_bounds__(kCompactThreads)
compact_kernel(uint4* k_cache, uint4* v_cache,     // read and written here: no __restrict__
               const uint4* __restrict__ new_k, const uint4* __restrict__ new_v,
               int len, int B, int N, const int32_t* __restrict__ kept_idx,
               const int32_t* __restrict__ first_evicted, int32_t* status) {
    __shared__ uint4 stage[kCompactRows * kRowVec];
    const int u = blockIdx.y;
    uint4* cache = blockIdx.x == 0 ? k_cache : v_cache;
    const uint4* block = blockIdx.x == 0 ? new_k : new_v;
    const int32_t* src_of = kept_idx + static_cast<size_t>(u) * N;
    // cache rows in front of the first evicted row stay; block rows (index >= len) always move
    for (int base = min(first_evicted[u], len); base < N; base += kCompactRows) {
        const int cnt = min(kCompactRows, N - base) * kRowVec;
        for (int q = threadIdx.x; q < cnt; q += kCompactThreads) {
            const int src = src_of[base + (q >> 4)];
            stage[q] = KD_ROW_OK(src, len + B, status) ? concat_row(cache, block, u, src, len, B, N)[q & 15] : make_uint4(0, 0, 0, 0);
        }
        __syncthreads();
        uint4* dst = cache + (static_cast<size_t>(u) * N + base) * kRowVec;
        for (int q = threadIdx.x; q < cnt; q += kCompactThreads) dst[q] = stage[q];
        __syncthreads();
    }
}

// Step a4 with unordered slot reuse (Eq. (keydiff) gathers the kept rows without fixing their order):
// kept cache rows stay where they are; the kept block rows, in block order, take the freed slots
// (evicted cache rows, then slots >= len that were still empty) in ascending slot order.  Input:
// kept[u][0..N) = ascending candidate numbers of the kept tokens (slots first, block rows after).
// Output: the rows, pos[u][slot] = token position, and kept[u][slot] rewritten to the candidate
// number each slot now holds.  grid = U, dynamic smem = 8 * B bytes.
__global__ void __launch_bounds__(kCompactThreads)
slot_place_kernel(uint4* __restrict__ k_cache, uint4* __restrict__ v_cache,
                  const uint4* __restrict__ new_k, const uint4* __restrict__ new_v,
                  int len, int B, int N, int32_t* __restrict__ kept, int32_t* __restrict__ pos, int next_pos,
                  unsigned long long* __restrict__ moved_rows) {
    extern __shared__ int32_t place[];   // slot_of[B], block_of[B]: the r-th freed slot, the r-th kept block row
    __shared__ int kc_sh;
    int32_t* slot_of = place;
    int32_t* block_of = place + B;
    const int u = blockIdx.x, tid = threadIdx.x;
    int32_t* L = kept + static_cast<size_t>(u) * N;
    // kc = kept cache rows = entries below len (L ascends): the one position where the list crosses len
    if (tid == 0) kc_sh = N;
    __syncthreads();
    for (int j = tid; j < N; j += kCompactThreads)
        if (L[j] >= len && (j == 0 || L[j - 1] < len)) kc_sh = j;
    __syncthreads();
    const int kc = kc_sh, kb = N - kc;   // kb kept block rows = kb freed slots
    for (int r = tid; r < kb; r += kCompactThreads) block_of[r] = L[kc + r] - len;
    // a slot s missing between L[j-1] and L[j] has j kept slots below it: it is freed slot number s - j
    for (int j = tid; j <= kc; j += kCompactThreads) {
        const int lo = j == 0 ? 0 : L[j - 1] + 1, hi = j == kc ? len : L[j];
        for (int sl = lo; sl < hi; ++sl) slot_of[sl - j] = sl;
    }
    for (int sl = len + tid; sl < N; sl += kCompactThreads) slot_of[sl - kc] = sl;   // the empty slots
    __syncthreads();
    for (int sl = tid; sl < N; sl += kCompactThreads) L[sl] = sl;
    __syncthreads();
    for (int r = tid; r < kb; r += kCompactThreads) {
        L[slot_of[r]] = len + block_of[r];
        pos[static_cast<size_t>(u) * N + slot_of[r]] = next_pos + block_of[r];
    }
    for (int q = tid; q < kb * kRowVec; q += kCompactThreads) {
        const int r = q >> 4, c = q & 15;
        const size_t dst = (static_cast<size_t>(u) * N + slot_of[r]) * kRowVec + c;
        const size_t src = (static_cast<size_t>(u) * B + block_of[r]) * kRowVec + c;
        k_cache[dst] = new_k[src];
        v_cache[dst] = new_v[src];
    }
    if (tid == 0) atomicAdd(moved_rows, static_cast<unsigned long long>(kb));
}

// Running anchor of the cached rows from the partial sums of anchor_partial_kernel run over the cache
// alone: sum[u][c] = sum over splits (double), and the pending deltas are cleared.  grid = U, 128 threads.
__global__ void anchor_fold_kernel(const double* __restrict__ partial, int splits, double* __restrict__ sum,
                                   double* __restrict__ delta, int ranks) {
    const int u = blockIdx.x, c = threadIdx.x;
    double a = 0.0;
    for (int s = 0; s < splits; ++s) a += partial[(static_cast<size_t>(u) * splits + s) * kHeadDim + c];
    sum[static_cast<size_t>(u) * kHeadDim + c] = a;
    for (int r = 0; r < ranks; ++r) delta[(static_cast<size_t>(u) * ranks + r) * kHeadDim + c] = 0.0;
}

// Token positions of the slots: identity (a cache the caller filled in token order) ...
__global__ void pos_iota_kernel(int32_t* __restrict__ pos, int N, int total) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < total) pos[i] = i % N;
}
// ... and those of appended block rows: slot len + j holds token next_pos + j.  grid = (ceil(B/threads), U).
__global__ void pos_append_kernel(int32_t* __restrict__ pos, int len, int B, int N, int next_pos) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j < B) pos[static_cast<size_t>(blockIdx.y) * N + len + j] = next_pos + j;
}

// Step a0 when the budget is not exceeded: rows [len, len+B) <- block rows, K and V.
// grid = (ceil(B*16/threads), U, 2).
__global__ void append_kernel(uint4* __restrict__ k_cache, uint4* __restrict__ v_cache,
                              const uint4* __restrict__ new_k, const uint4* __restrict__ new_v,
                              int len, int B, int N) {
    const int u = blockIdx.y;
    uint4* cache = blockIdx.z == 0 ? k_cache : v_cache;
    const uint4* block = blockIdx.z == 0 ? new_k : new_v;
    const int q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q < B * kRowVec)
        cache[(static_cast<size_t>(u) * N + len) * kRowVec + q] = block[static_cast<size_t>(u) * B * kRowVec + q];
}

}  // namespace kd
