// The eviction step with unordered slot reuse as one streaming kernel.
//
// Eq. (keydiff) gathers the kept rows, K' = gather(K, S), without fixing their order, and attention does
// not depend on the order of the cached pairs.  With slot reuse the kept cache rows stay where they are
// and the kept block rows are written into the freed slots, so the step only has to READ the unit's keys
// once (to score them, App. B.1) and to write at most B rows of K and V.  Nothing has to stay on chip:
// a cluster of C CTAs (C may be 1) streams its unit's K rows through a ring of 16-row tiles in shared
// memory, warp w owning ring slots w, w+16, ...: it waits for a tile, scores its rows against the anchor
// (known beforehand from the running sum, see fused_kernel.cuh), and at once refills the slot with the
// next tile of its stream, which runs on into the cluster's next unit.  The loads of a unit therefore
// arrive while the previous unit is being selected.
//
//   anchor   running sum + deltas + the block rows' terms (every CTA normalises the whole block)
//   scores   per tile as it lands; keys into the CTA's table; the slice's keys pushed to the peers (DSMEM)
//   select   every CTA on its own full copy of the table (the low-end select of fused_kernel.cuh, or the
//            full-table select); result: the bitmap of evicted candidates, the same in every CTA
//   place    from the bitmap every CTA derives the same three lists (evicted candidates, freed slots,
//            kept block rows); row group number r of the cluster reads evicted row r once more (its
//            k/||k|| leaves the running sum) and writes kept block row r into freed slot r
//
// One cluster barrier per unit (all keys delivered) plus a split one that keeps a peer's next push away
// from a table still being read; none when C = 1.  Every wait is bounded (status word on expiry).
#pragma once
#include "fused_kernel.cuh"

namespace kd {

constexpr int kSlotMaxRing = 3 * kFusedWarps;   // at most three tiles per warp in the ring
constexpr int kSlotMaxBlock = 1024;   // the three lists of a step live in shared memory, max_block entries each

struct SlotLayout {
    int ring, keys, work, bitmap, cand, lists, sel, mu, mbar, misc, total;
};
__host__ __device__ inline SlotLayout slot_layout(int ring_tiles, int nkeys, int nwords, int max_block) {
    SlotLayout L;
    int off = 0;
    auto take = [&off](int bytes) { const int o = off; off += (bytes + 127) & ~127; return o; };
    // fixed-size regions first: compile-time addresses (the ring's too), which keeps them out of the registers
    L.misc = take(128);
    L.mbar = take(kSlotMaxRing * 8);
    L.mu = take(kHeadDim * 4);
    L.sel = take(static_cast<int>(sizeof(SelectSmem)));
    L.cand = take(2 * kCandCap * 4);     // keys and indices of the threshold bin
    L.work = take(kBins * 4);            // warp-reduction scratch / histogram
    L.ring = take(ring_tiles * kTileRows * kRowBytes);
    L.keys = take(nkeys * 4 > kReduceBytes ? nkeys * 4 : kReduceBytes);   // also the reduction scratch while the table is dead
    L.bitmap = take(2 * nwords * 4);     // evicted-candidate bitmap, evicted-before count of every word
    L.lists = take(3 * max_block * 4);   // evicted candidates, freed slots, kept block rows
    L.total = off;
    return L;
}

struct SlotParams {
    uint4* k_cache; uint4* v_cache; const uint4* new_k; const uint4* new_v;
    int len, B, N, U;
    float eps;
    int cluster;        // CTAs per cluster
    int rows_per_cta;   // slice length, a multiple of kTileRows
    int ring_tiles;     // tiles in the ring, a multiple of the warp count
    int nkeys;          // key-table capacity (>= cluster * rows_per_cta)
    int nwords;         // bitmap words provided for (>= ceil(n / 32))
    int nmax;           // row stride of the score scratch
    int max_block;
    unsigned stagger_ns;   // cluster c starts c * stagger_ns late
    unsigned late_ns;      // clusters that serve one unit fewer than the others start this much later still
    float* scores; int32_t* kept_idx; int32_t* first_evicted;
    unsigned long long* moved_rows; int32_t* status;
    const double* anchor_in; double* anchor_out; double* anchor_delta;   // running anchor, as in FusedParams
    int raw_anchor, window;
    int32_t* pos;       // [U][N] token position of every slot
    int next_pos;       // position of the block's first token
    int32_t* kept_mirror;   // optional second destination of the slot list (device alias of pinned host memory)
};

// One thread: bulk-load unit rows [g0, g0 + nrows) of unit u (cache rows below len, block rows after) to dst.
__device__ __forceinline__ void issue_rows(const uint4* cache, const uint4* block, int u, int len, int B, int N,
                                           int g0, int nrows, uint32_t dst, uint32_t bar) {
    const int from_cache = min(max(len - g0, 0), nrows);
    const int from_block = nrows - from_cache;
    mbar_expect_tx(bar, nrows * kRowBytes);
    if (from_cache > 0)
        bulk_load(dst, cache + (static_cast<size_t>(u) * N + g0) * kRowVec, from_cache * kRowBytes, bar);
    if (from_block > 0)
        bulk_load(dst + from_cache * kRowBytes,
                  block + (static_cast<size_t>(u) * B + (g0 + from_cache - len)) * kRowVec, from_block * kRowBytes, bar);
}

__global__ void __launch_bounds__(kFusedThreads, 1) slot_evict_kernel(const SlotParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int C = p.cluster;
    const SlotLayout L = slot_layout(p.ring_tiles, p.nkeys, p.nwords, p.max_block);
    const uint4* ring = reinterpret_cast<const uint4*>(smem + L.ring);
    uint32_t* keys = reinterpret_cast<uint32_t*>(smem + L.keys);
    int* hist = reinterpret_cast<int*>(smem + L.work);
    uint32_t* bitmap = reinterpret_cast<uint32_t*>(smem + L.bitmap);
    int* wlocal = reinterpret_cast<int*>(smem + L.bitmap) + p.nwords;
    uint32_t* cand_key = reinterpret_cast<uint32_t*>(smem + L.cand);
    int* cand_idx = reinterpret_cast<int*>(smem + L.cand) + kCandCap;
    int* ev_of = reinterpret_cast<int*>(smem + L.lists);   // evicted candidates, ascending
    int* slot_of = ev_of + p.max_block;                    // freed slots, ascending
    int* blk_of = slot_of + p.max_block;                   // kept block rows, ascending
    SelectSmem& sel = *reinterpret_cast<SelectSmem*>(smem + L.sel);
    float* mu_sh = reinterpret_cast<float*>(smem + L.mu);
    int* misc = reinterpret_cast<int*>(smem + L.misc);   // 0 ncand, 1 first evicted, 2 need_eq, 3 threshold key, 5/6 prefix carry, 12 a wait ran out
    const uint32_t ring_sa = smem_addr(ring), mbar_sa = smem_addr(smem + L.mbar), keys_sa = smem_addr(keys);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = tid >> 3, t = tid & 7, sub = lane >> 3;
    const int crank = static_cast<int>(cluster_ctarank());
    const int cluster_id = blockIdx.x / C, nclusters = gridDim.x / C;
    const int len = p.len, B = p.B, N = p.N, n = len + B, E = n - N;   // E candidates are evicted
    const float inv_eps = 1.0f / p.eps;
    const bool raw = p.raw_anchor != 0;
    const int nwords = (n + 31) >> 5;
    const int seg_a = min(n, crank * p.rows_per_cta);
    const int seg = min(n, seg_a + p.rows_per_cta) - seg_a, seg_b = seg_a + seg;
    // The slice as a stream of 16-row tiles; warp w takes tiles w, w+16, ... of every unit of the cluster,
    // one unit after the other, through its own D ring slots (slot w + 16 d).
    const int nvt = (seg + kTileRows - 1) / kTileRows;
    const int cnt_w = warp < nvt ? (nvt - warp + kFusedWarps - 1) / kFusedWarps : 0;   // tiles per unit for this warp
    const int D = p.ring_tiles / kFusedWarps;
    const int my_units = cluster_id < p.U ? (p.U - cluster_id + nclusters - 1) / nclusters : 0;

    if (tid == 0) {
        for (int j = 0; j < p.ring_tiles; ++j) mbar_init(mbar_sa + 8 * j, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        misc[12] = 0;
    }
    __syncthreads();
    if (p.stagger_ns != 0 && cluster_id != 0) {   // bounded start-up delay that spreads the clusters' phases
        const unsigned long long t0 = global_timer_ns();
        const unsigned long long wait_ns = static_cast<unsigned long long>(p.stagger_ns) * static_cast<unsigned>(cluster_id);
        for (int spin = 0; spin < (1 << 16) && global_timer_ns() - t0 < wait_ns; ++spin) __nanosleep(100);
    }
    // When the units do not divide evenly, the clusters with one unit fewer have a unit's time to spare: they
    // start late, so that their stream runs while the others are between streams (selection, placement)
    // instead of competing with the others' first stream.  Bounded like the wait above.
    if (p.late_ns != 0 && my_units > 0 && my_units < (p.U + nclusters - 1) / nclusters) {
        const unsigned long long t0 = global_timer_ns();
        for (int spin = 0; spin < (1 << 16) && global_timer_ns() - t0 < p.late_ns; ++spin) __nanosleep(200);
    }

    // issue side of the warp's stream: the next tile to request is tile i_j of the cluster's i_it-th unit
    int i_it = 0, i_j = 0;
    auto issue_next = [&](int d) {   // lane 0 only; d = ring slot (of this warp) to fill
        const int vt = warp + kFusedWarps * i_j;
        const int lo = vt * kTileRows, hi = min(seg, lo + kTileRows);
        const int phys = warp + kFusedWarps * d;
        issue_rows(p.k_cache, p.new_k, cluster_id + i_it * nclusters, len, B, N, seg_a + lo, hi - lo,
                   ring_sa + phys * kTileRows * kRowBytes, mbar_sa + 8 * phys);
        if (++i_j == cnt_w) { i_j = 0; ++i_it; }
    };
    if (lane == 0 && cnt_w > 0)
        for (int d = 0; d < D && i_it < my_units; ++d) issue_next(d);
    int c_d = 0;            // ring slot the next tile of the stream arrives in
    uint32_t c_par = 0;     // bit d: parity the next wait on slot d expects
    bool exchange_pending = false;   // an arrive of the split cluster barrier has no wait yet

    for (int u = cluster_id; u < p.U; u += nclusters) {
        const int un = u + nclusters;
        double block_sum = 0.0;   // tid < 128: channel tid of the block rows' sum of k/||k||
        // ------------------------------------------------------------ anchor from the running sum + the block rows
        {
            double run = 0.0;
            double dl[kMaxCluster];
            if (tid < kHeadDim) {
                run = p.anchor_in[static_cast<size_t>(u) * kHeadDim + tid];
#pragma unroll
                for (int c = 0; c < kMaxCluster; ++c)
                    dl[c] = c < C ? p.anchor_delta[(static_cast<size_t>(u) * C + c) * kHeadDim + tid] : 0.0;
            }
            // every CTA normalises the whole block itself, one warp per row (the canonical form of a row's terms, see
            // fused_kernel.cuh), eight rows requested at a time; scratch: the work area (the key table cannot lend its
            // space here: a peer that is ahead may already be pushing its keys of this unit into it)
            {
                const uint4* blk = p.new_k + static_cast<size_t>(u) * B * kRowVec;
                double acc[4] = {0.0, 0.0, 0.0, 0.0};
                for (int j0 = warp; j0 < B; j0 += 8 * kFusedWarps) {   // (warp-uniform)
                    uint2 wds[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const int j = j0 + k * kFusedWarps;
                        wds[k] = j < B ? reinterpret_cast<const uint2*>(blk + static_cast<size_t>(j) * kRowVec)[lane] : make_uint2(0, 0);
                    }
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        if (j0 + k * kFusedWarps < B) warp_row_terms(wds[k], true, inv_eps, raw, acc);
                }
                block_sum = cta_sum_of_warp_sums(acc, reinterpret_cast<double*>(smem + L.work), tid);
            }
            if (tid < kHeadDim) {
                double a = run;
#pragma unroll
                for (int c = 0; c < kMaxCluster; ++c) a += dl[c];   // rank order; absent ranks add 0
                if (crank == 0) p.anchor_out[static_cast<size_t>(u) * kHeadDim + tid] = a;   // the cached rows' sum, folded
                mu_sh[tid] = static_cast<float>((a + block_sum) / static_cast<double>(n));
            }
            __syncthreads();
        }
        // ------------------------------------------------------------ a1 + a2 in one pass over the stream
        {
            float2 w[8];
            load_anchor(mu_sh, t, w);
            float m;   // ||mu||, computed by every warp in the same order
            {
                const float4 c4 = reinterpret_cast<const float4*>(mu_sh)[lane];
                float v = fmaf(c4.w, c4.w, fmaf(c4.z, c4.z, fmaf(c4.y, c4.y, c4.x * c4.x)));
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                m = sqrtf(v);
            }
            float* sc = p.scores + static_cast<size_t>(u) * p.nmax + seg_a;
#pragma unroll 1
            for (int j = 0; j < cnt_w; ++j) {
                const int phys = warp + kFusedWarps * c_d;
                // (a tile that never landed: from then on this CTA places no row and reports no change to the running sum)
                if (!mbar_wait(mbar_sa + 8 * phys, (c_par >> c_d) & 1u, p.status)) misc[12] = 1;
                c_par ^= 1u << c_d;
                const int lo = (warp + kFusedWarps * j) * kTileRows;   // first slice row of the tile
                const uint4* tile = ring + phys * kTileRows * kRowVec;
                float vs[4];   // this lane's shares of the tile's four rows of its row group
                double vd[4];
#pragma unroll
                for (int it = 0; it < 4; ++it) {
                    const int r = it * 4 + sub;
                    uint4 a = make_uint4(0, 0, 0, 0), b = a;
                    if (lo + r < seg) { a = tile[r * kRowVec + t]; b = tile[r * kRowVec + t + 8]; }
                    lane_sumsq_dot(a, b, w, vs[it], vd[it]);
                }
                const uint32_t key = score4(vs, vd, t, m, p.eps);
                const int lr = lo + (t >> 1) * 4 + sub;
                if (!(t & 1) && lr < seg) {
                    keys[seg_a + lr] = key;
                    sc[lr] = key_score(key);   // fp32 score to global scratch: the tile's 16 scores are one 64-byte line
                }
                __syncwarp();   // the tile's only readers are this warp's lanes: the copy engine may refill it
                if (lane == 0 && i_it < my_units) issue_next(c_d);
                if (++c_d == D) c_d = 0;
            }
        }
        if (exchange_pending) { cluster_wait(); exchange_pending = false; }   // the peers are done with the previous unit's table
        __syncthreads();
        if (C > 1) {
            // this slice's keys -> every peer's table (128-bit DSMEM stores; slices are multiples of 16 rows)
            const uint4* mine = reinterpret_cast<const uint4*>(keys + seg_a);
            for (int c = 1; c < C; ++c) {
                const int peer = crank + c < C ? crank + c : crank + c - C;
                const uint32_t base = map_to_cta(keys_sa + 4 * seg_a, peer);
                for (int o = tid; 4 * o < seg; o += kFusedThreads) st_cluster_v4(base + 16 * o, mine[o]);
            }
            cluster_arrive();
        }
        {
            for (int b = tid; b < kBins; b += kFusedThreads) hist[b] = 0;
            for (int wd = tid; wd < nwords; wd += kFusedThreads) bitmap[wd] = 0;
            if (tid == 0) { misc[0] = 0; misc[1] = n; }
        }
        if (C > 1) cluster_wait();   // (2) the key table of every CTA holds all n keys
        __syncthreads();
        if (p.window > 0) {
            // sliding window (Sec. 3.2): tokens at the last `window` positions of the sequence get the largest
            // possible key, so they are never among the E smallest
            const int first_recent = p.next_pos + B - p.window;
            for (int i = len + max(B - p.window, 0) + tid; i < n; i += kFusedThreads) keys[i] = 0xffffffffu;
            if (p.window > B) {
                const int32_t* ps = p.pos + static_cast<size_t>(u) * N;
                for (int i = tid; i < len; i += kFusedThreads) if (ps[i] >= first_recent) keys[i] = 0xffffffffu;
            }
            __syncthreads();
        }
        // ------------------------------------------------------------ a3: the bitmap of evicted candidates
        // the low-end select of fused_kernel.cuh; ties: (key ascending, candidate number descending) go first
        int* wbase = sel.hist + 2 * kFusedWarps;
        const bool planned = low_end_select(keys, n, E, hist, bitmap, cand_key, cand_idx, sel, misc);
        if (!planned) {
            // the full-table select writes the same bitmap (cleared first: the attempt above may have marked some)
            for (int wd = tid; wd < nwords; wd += kFusedThreads) bitmap[wd] = 0;
            __syncthreads();
            full_select_plan(keys, n, N, 0, 0, hist, cand_key, cand_idx, nullptr, sel, misc, bitmap);
        }
        {
            // evicted candidates before each word of the bitmap
            for (int w0 = 0; w0 < nwords; w0 += kFusedThreads) {   // (nwords <= 512 on the low-end route; any size here)
                const int wi = w0 + tid;
                const int pc = wi < nwords ? __popc(bitmap[wi]) : 0;
                int incl = pc;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int v = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += v;
                }
                if (wi < nwords) wlocal[wi] = incl - pc;   // within its warp's 32 words
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
                if (wi < nwords) wlocal[wi] += wbase[warp];   // evicted candidates before word wi
                if (tid == 0) misc[5] = misc[6];
                __syncthreads();
            }
        }
        auto evicted_before = [&](int i) { const int w = i >> 5; return wlocal[w] + __popc(bitmap[w] & ((1u << (i & 31)) - 1u)); };
        // ------------------------------------------------------------ the three lists, the same in every CTA
        const int evicted_cache = evicted_before(len);   // evicted candidates among the len cache slots (len < n)
        const int kept_cache = len - evicted_cache;
        const int kb = N - kept_cache;                   // kept block rows = freed slots
        for (int w = tid; w < nwords; w += kFusedThreads) {
            int e = wlocal[w];
            for (uint32_t wd = bitmap[w]; wd; wd &= wd - 1) {
                const int i = 32 * w + __ffs(wd) - 1;
                ev_of[e] = i;
                if (i < len) slot_of[e] = i;   // every candidate before a cache slot is a cache slot
                ++e;
            }
        }
        for (int j = tid; j < B; j += kFusedThreads) {
            const int i = len + j;
            if (!((bitmap[i >> 5] >> (i & 31)) & 1u)) blk_of[(i - evicted_before(i)) - kept_cache] = j;
        }
        for (int e = len + tid; e < N; e += kFusedThreads) slot_of[evicted_cache + (e - len)] = e;   // slots that were still empty
        // kept cache rows of this slice keep their slot: the kept-index list says so
        for (int i = seg_a + tid; i < min(seg_b, len); i += kFusedThreads)
            if (!((bitmap[i >> 5] >> (i & 31)) & 1u)) {
                p.kept_idx[static_cast<size_t>(u) * N + i] = i;
                if (p.kept_mirror) p.kept_mirror[static_cast<size_t>(u) * N + i] = i;
            }
        if (crank == 0 && tid == 0) {
            p.first_evicted[u] = misc[1];
            atomicAdd(p.moved_rows, static_cast<unsigned long long>(kb));
        }
        if (crank == 0 && un < p.U) {   // the next unit's block rows towards L2: every CTA reads them first thing
            const char* nb = reinterpret_cast<const char*>(p.new_k + static_cast<size_t>(un) * B * kRowVec);
            for (int o = tid * 128; o < B * kRowBytes; o += kFusedThreads * 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(nb + o));
        }
        __syncthreads();
        // ------------------------------------------------------------ a4: evicted rows leave the running sum, kept block rows take the freed slots
        {
            // (a) evicted rows, read once more (from L2): their terms leave the running sum.  The CTA that re-reads
            // evicted row r is the one that overwrites its slot in (b): rows r with (r / 64) % C == crank.
            const int stride = C * kGroups, r_first = crank * kGroups + g;
            {
                const int rem = E % stride - crank * kGroups;
                const int mine = (E / stride) * kGroups + min(max(rem, 0), kGroups);
                double acc[4] = {0.0, 0.0, 0.0, 0.0};
                for (int j0 = warp; j0 < mine; j0 += 8 * kFusedWarps) {   // one warp per row, eight rows requested at a time
                    uint2 wds[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const int j = j0 + k * kFusedWarps;
                        wds[k] = make_uint2(0, 0);
                        if (j < mine) {
                            const int v = ev_of[(j / kGroups) * stride + crank * kGroups + (j % kGroups)];
                            // (an entry outside [0, n) cannot occur; the clamp makes sure that even then no address
                            // outside the tensors is formed)
                            wds[k] = reinterpret_cast<const uint2*>(concat_row(p.k_cache, p.new_k, u, min(max(v, 0), n - 1), len, B, N))[lane];
                        }
                    }
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        if (j0 + k * kFusedWarps < mine) warp_row_terms(wds[k], true, inv_eps, raw, acc);
                }
                const double gone = cta_sum_of_warp_sums(acc, reinterpret_cast<double*>(keys), tid);   // the key table is dead until the next unit
                if (tid < kHeadDim)
                    p.anchor_delta[(static_cast<size_t>(u) * C + crank) * kHeadDim + tid] = misc[12] == 0 ? (crank == 0 ? block_sum : 0.0) - gone : 0.0;
                // (the barriers inside the sum lie behind every read of an evicted row: its slot may be overwritten)
            }
            // (b) kept block row r into freed slot r.  For r < evicted_cache that slot is evicted row r, which this
            // same CTA re-read in (a), in front of the barrier above.
#pragma unroll 2
            for (int r = misc[12] == 0 ? r_first : kb; r < kb; r += stride) {
                const int slot = slot_of[r], j = blk_of[r];
                const uint4* sk = p.new_k + (static_cast<size_t>(u) * B + j) * kRowVec;
                const uint4* sv = p.new_v + (static_cast<size_t>(u) * B + j) * kRowVec;
                uint4* dk = p.k_cache + (static_cast<size_t>(u) * N + slot) * kRowVec;
                uint4* dv = p.v_cache + (static_cast<size_t>(u) * N + slot) * kRowVec;
                const uint4 k0 = sk[t], k1 = sk[t + 8], v0 = sv[t], v1 = sv[t + 8];
                if (!(KD_ROW_OK(slot, N, p.status) && KD_ROW_OK(j, B, p.status))) continue;
                dk[t] = k0; dk[t + 8] = k1;
                dv[t] = v0; dv[t + 8] = v1;
                if (t == 0) {
                    p.kept_idx[static_cast<size_t>(u) * N + slot] = len + j;
                    if (p.kept_mirror) p.kept_mirror[static_cast<size_t>(u) * N + slot] = len + j;
                    p.pos[static_cast<size_t>(u) * N + slot] = p.next_pos + j;
                }
            }
        }
        if (C > 1) { cluster_arrive(); exchange_pending = true; }   // this CTA is done with the unit's key table
        __syncthreads();   // the scratch areas are free for the next unit
    }
    if (exchange_pending) cluster_wait();
    if (C > 1) cluster_sync_all();   // no CTA leaves while a peer may still address its shared memory
}

}  // namespace kd
