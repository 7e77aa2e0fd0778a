// Shared device helpers of libbz: order keys, the vote on bit patterns, launch bookkeeping.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/bz.h"

namespace bz {

constexpr int kNumSMs = 148;  // B200: 2 dies x 74 SMs; grids are sized in multiples of this

// ---- host-side bookkeeping -----------------------------------------------------------------
void note_launch();                       // counts one kernel launch
int cuda_failed(cudaError_t e);           // records the message, returns BZ_ERR_CUDA
int check_launch();                       // cudaGetLastError() after a launch -> status
void note_path(int path);                 // which kernel family a call dispatched to (BZ_PATH_*), per host thread

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned8(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 7u) == 0; }
inline bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- IEEE total order as a signed 32-bit key ------------------------------------------------
// Negative patterns get their 31 magnitude bits flipped, so signed integer comparison of keys is
// the total order  -NaN < -inf < ... < -0 < +0 < ... < +inf < +NaN.  The map is its own inverse.
__device__ __forceinline__ int order_key(uint32_t bits) {
    const int x = static_cast<int>(bits);
    return x ^ ((x >> 31) & 0x7fffffff);
}
__device__ __forceinline__ uint32_t key_bits(int key) { return static_cast<uint32_t>(key ^ ((key >> 31) & 0x7fffffff)); }

__device__ __forceinline__ int kmin(int a, int b) { return min(a, b); }
__device__ __forceinline__ int kmax(int a, int b) { return max(a, b); }
// binary32 comparators for columns of finite values (numeric order = total order up to the sign of zeros, which no
// result depends on).  A NaN comes out of BOTH sides, so that it reaches the ends of a sorted column, where the
// caller looks for it.
__device__ __forceinline__ float kmin(float a, float b) {
    float m;
    asm("min.NaN.f32 %0, %1, %2;" : "=f"(m) : "f"(a), "f"(b));
    return m;
}
__device__ __forceinline__ float kmax(float a, float b) {
    float m;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(m) : "f"(a), "f"(b));
    return m;
}

// Integer min/max issue on the ALU pipe (64 lanes per SM and clock) while the multiply-add pipe idles in a
// comparator network.  max = a + b - min (exact modulo 2^32) as two integer multiply-adds moves one of a
// comparator's two operations there; the multipliers are read from constant memory so that the compiler
// cannot fold them into an addition (which would issue on the ALU pipe again).  A loop of comparators alone
// runs 26 % faster with every other comparator done this way; a network's run<NUM, DEN> does it for NUM of
// every DEN full comparators, and only kernels bound by the ALU pipe ask for it.
static __constant__ unsigned int kPipeOne = 1u, kPipeMinusOne = 0xffffffffu;
#define BZ_CE(a, b, i)                                                                                            \
    {                                                                                                             \
        const T lo_ = kmin(k[a], k[b]);                                                                           \
        if constexpr (((i) % DEN) < NUM)                                                                          \
            k[b] = static_cast<T>(static_cast<unsigned int>(lo_) * kPipeMinusOne +                                \
                                  (static_cast<unsigned int>(k[a]) * kPipeOne + static_cast<unsigned int>(k[b]))); \
        else                                                                                                      \
            k[b] = kmax(k[a], k[b]);                                                                              \
        k[a] = lo_;                                                                                               \
    }
#define BZ_LO(a, b) k[a] = kmin(k[a], k[b]);
#define BZ_HI(a, b) k[b] = kmax(k[a], k[b]);

template <int N> struct MedianNet;  // specialisations in sort_networks.inc
template <int N> struct SortNet;
#include "sort_networks.inc"

// ---- Eq. (3) on one coordinate ---------------------------------------------------------------
// Plurality of R bit patterns; among equally frequent patterns the first seen wins.
template <int R> __device__ __forceinline__ uint32_t vote_bits(const uint32_t (&x)[R]) {
    if constexpr (R == 1) {
        return x[0];
    } else if constexpr (R == 3) {
        return (x[1] == x[2]) ? x[1] : x[0];
    } else {
        // A pattern held by more than half of the copies is the winner whatever the order, and it shows up among
        // any R/2 + 1 copies.  Honest copies are identical, so copy 0 wins at once unless it is a Byzantine one;
        // then the next R/2 copies are tried together, without branches.
        constexpr int kHalf = R / 2 + 1;
        int same0 = 1;
#pragma unroll
        for (int k = 1; k < R; ++k) same0 += (x[k] == x[0]);
        if (same0 >= kHalf) return x[0];
        uint32_t major = x[0];
        bool found = false;
#pragma unroll
        for (int c = kHalf - 1; c >= 1; --c) {
            int same = 0;
#pragma unroll
            for (int k = 0; k < R; ++k) same += (x[k] == x[c]);
            const bool hit = same >= kHalf;
            major = hit ? x[c] : major;
            found = found || hit;
        }
        if (found) return major;
        // no majority: plurality, the pattern first seen wins among equally frequent ones
        uint32_t best = x[0];
        int best_count = same0;
#pragma unroll
        for (int k = 1; k < R; ++k) {
            int count = 0;
#pragma unroll
            for (int k2 = 0; k2 < R; ++k2) count += (x[k2] == x[k]);
            if (count > best_count) {
                best_count = count;
                best = x[k];
            }
        }
        return best;
    }
}

// Run-time r (generic path): same rule on an array in local memory.
__device__ __forceinline__ uint32_t vote_bits_dyn(const uint32_t* x, int r) {
    uint32_t best = x[0];
    int best_count = 0;
    for (int k = 0; k < r; ++k) {
        int count = 0;
        for (int k2 = 0; k2 < r; ++k2) count += (x[k2] == x[k]);
        if (count > best_count) {
            best_count = count;
            best = x[k];
        }
    }
    return best;
}

// ---- Eq. (1): the model update, applied where an aggregate is produced -------------------------
// w == nullptr means "no update".  With a velocity buffer: v <- mu*v + g, w <- w - eta*v (one
// fused multiply-add each); without: w <- w - eta*g.
struct ModelUpdate {
    float* w;
    float* v;
    float eta, mu;
};
__device__ __forceinline__ float update_lane(float w, float& v, float g, float eta, float mu, bool has_v) {
    float step = g;
    if (has_v) {
        v = __fmaf_rn(mu, v, g);
        step = v;
    }
    return __fmaf_rn(-eta, step, w);
}
__device__ __forceinline__ void apply_update(const ModelUpdate& u, int64_t j, float g) {
    float v = 0.f;
    const bool has_v = u.v != nullptr;
    if (has_v) v = u.v[j];
    u.w[j] = update_lane(u.w[j], v, g, u.eta, u.mu, has_v);
    if (has_v) u.v[j] = v;
}
// four consecutive coordinates starting at 4*j4 (w and v 16-byte aligned)
__device__ __forceinline__ void apply_update4(const ModelUpdate& u, int64_t j4, const uint4& gbits) {
    const bool has_v = u.v != nullptr;
    float4 w = reinterpret_cast<float4*>(u.w)[j4];
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (has_v) v = reinterpret_cast<float4*>(u.v)[j4];
    w.x = update_lane(w.x, v.x, __uint_as_float(gbits.x), u.eta, u.mu, has_v);
    w.y = update_lane(w.y, v.y, __uint_as_float(gbits.y), u.eta, u.mu, has_v);
    w.z = update_lane(w.z, v.z, __uint_as_float(gbits.z), u.eta, u.mu, has_v);
    w.w = update_lane(w.w, v.w, __uint_as_float(gbits.w), u.eta, u.mu, has_v);
    reinterpret_cast<float4*>(u.w)[j4] = w;
    if (has_v) reinterpret_cast<float4*>(u.v)[j4] = v;
}

// ---- streaming loads (read-once data: evict-first) -------------------------------------------
__device__ __forceinline__ uint4 ld_stream(const uint4* p) { return __ldcs(p); }
__device__ __forceinline__ uint2 ld_stream(const uint2* p) { return __ldcs(p); }
__device__ __forceinline__ uint32_t ld_stream(const uint32_t* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(uint4* p, const uint4& x) { __stcs(p, x); }
__device__ __forceinline__ void st_stream(uint2* p, const uint2& x) { __stcs(p, x); }
__device__ __forceinline__ void st_stream(uint32_t* p, uint32_t x) { __stcs(p, x); }

}  // namespace bz
