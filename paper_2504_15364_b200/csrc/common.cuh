// Device helpers shared by the KeyDiff kernels (sm_100a).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace kd {

constexpr int kHeadDim = 128;              // channels per key/value row
constexpr int kRowBytes = kHeadDim * 2;    // bf16 row = 256 B
constexpr int kRowVec = kRowBytes / 16;    // 16 x 128-bit words per row
constexpr int kLanesPerRow = 8;            // a row is handled by 8 consecutive lanes

// Debug build (-DKEYDIFF_DEBUG_CHECKS, see build.py --debug-checks): every destination row index a kernel computes
// is range-checked before the store; a bad index is recorded in the status word (KEYDIFF_ERR_INTERNAL) and the
// store is skipped.  Without the macro the check is not compiled.
constexpr int kErrInternal = -8;   // KEYDIFF_ERR_INTERNAL
#ifdef KEYDIFF_DEBUG_CHECKS
#define KD_ROW_OK(d, limit, status) ((static_cast<unsigned>(d) < static_cast<unsigned>(limit)) || (atomicExch((status), kd::kErrInternal), false))
#else
#define KD_ROW_OK(d, limit, status) true
#endif

// bf16 is the upper half of a binary32: widening is a shift / a mask.
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Lane t (0..7) of a row group owns 128-bit words t and t+8 of the row, i.e. channels
// [8t, 8t+8) and [64+8t, 64+8t+8): consecutive lanes read consecutive 16-byte words, so
// a row group's load is one contiguous 128-byte segment (coalesced in global memory,
// conflict-free in shared memory).
__device__ __forceinline__ void unpack_row(const uint4& a, const uint4& b, float (&x)[16]) {
    x[0] = bf16_lo(a.x); x[1] = bf16_hi(a.x); x[2] = bf16_lo(a.y); x[3] = bf16_hi(a.y);
    x[4] = bf16_lo(a.z); x[5] = bf16_hi(a.z); x[6] = bf16_lo(a.w); x[7] = bf16_hi(a.w);
    x[8] = bf16_lo(b.x); x[9] = bf16_hi(b.x); x[10] = bf16_lo(b.y); x[11] = bf16_hi(b.y);
    x[12] = bf16_lo(b.z); x[13] = bf16_hi(b.z); x[14] = bf16_lo(b.w); x[15] = bf16_hi(b.w);
}

// channel index of register j (0..15) of lane t
__device__ __forceinline__ int lane_channel(int t, int j) { return (j < 8 ? 8 * t : 64 + 8 * t) + (j & 7); }

// sum over the 8 lanes of a row group (xor butterflies stay inside an aligned group of 8)
__device__ __forceinline__ float group_sum(float v) {
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    v += __shfl_xor_sync(0xffffffffu, v, 2);
    v += __shfl_xor_sync(0xffffffffu, v, 4);
    return v;
}

// Sum of squares of a lane's 16 channels, then over the row group: ||k||^2 in fp32.
__device__ __forceinline__ float row_sumsq(const float (&x)[16]) {
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) { s0 = fmaf(x[j], x[j], s0); s1 = fmaf(x[8 + j], x[8 + j], s1); }
    return group_sum(s0 + s1);
}

// mu.k over the row group.  Products and chains of four of them are fp32 (a product of a bf16 value and an
// fp32 value rounds at the size of that one term); everything above them -- the four chains of a lane and
// the eight lanes of the group -- is added in double precision, because a cosine near zero is a sum of
// terms that cancel and fp32 partial sums of the size of the terms would decide its last digits.
__device__ __forceinline__ double group_sum(double v) {
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    v += __shfl_xor_sync(0xffffffffu, v, 2);
    v += __shfl_xor_sync(0xffffffffu, v, 4);
    return v;
}
__device__ __forceinline__ float row_dot(const float (&x)[16], const float (&w)[16]) {
    float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        c[0] = fmaf(x[j], w[j], c[0]); c[1] = fmaf(x[4 + j], w[4 + j], c[1]);
        c[2] = fmaf(x[8 + j], w[8 + j], c[2]); c[3] = fmaf(x[12 + j], w[12 + j], c[3]);
    }
    const double lane = (static_cast<double>(c[0]) + static_cast<double>(c[1])) + (static_cast<double>(c[2]) + static_cast<double>(c[3]));
    return static_cast<float>(group_sum(lane));
}

// App. B.1, second expression, then the eviction score e = -s with -0 mapped to +0.
__device__ __forceinline__ float eviction_score(float dot, float anchor_norm, float key_norm, float eps) {
    const float s = dot / fmaxf(anchor_norm * key_norm, eps);
    const float e = -s;
    return e == 0.f ? 0.f : e;
}

// Monotone map fp32 -> u32: a < b  <=>  key(a) < key(b)  (for non-NaN values).
__device__ __forceinline__ uint32_t order_key(float e) {
    const uint32_t u = __float_as_uint(e);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

}  // namespace kd
