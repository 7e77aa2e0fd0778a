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

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
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

#define BZ_CE(a, b)                         \
    {                                       \
        const T lo_ = kmin(k[a], k[b]);     \
        k[b] = kmax(k[a], k[b]);            \
        k[a] = lo_;                         \
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
        int same0 = 1;
#pragma unroll
        for (int k = 1; k < R; ++k) same0 += (x[k] == x[0]);
        if (2 * same0 >= R) return x[0];  // nothing can be strictly more frequent than copy 0
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

// ---- streaming loads (read-once data: evict-first) -------------------------------------------
__device__ __forceinline__ uint4 ld_stream(const uint4* p) { return __ldcs(p); }
__device__ __forceinline__ uint32_t ld_stream(const uint32_t* p) { return __ldcs(p); }

}  // namespace bz
