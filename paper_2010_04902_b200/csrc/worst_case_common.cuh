// Pieces shared by the two exhaustive searches: bit-sliced holder counts, the running best and its
// reduction over a block and over the grid.
#pragma once

#include "bz_common.cuh"

namespace bz {

constexpr int kWcBlock = 128;
constexpr int kWcMaxBlocks = kNumSMs * 12;

struct Planes {
    uint64_t c0, c1, c2;
};

__device__ __forceinline__ Planes add_mask(const Planes& s, uint64_t m) {
    Planes o;
    o.c0 = s.c0 ^ m;
    const uint64_t k0 = s.c0 & m;
    o.c1 = s.c1 ^ k0;
    const uint64_t k1 = s.c1 & k0;
    o.c2 = s.c2 ^ k1;
    return o;
}

// files with at least RP holders
template <int RP> __device__ __forceinline__ int count_at_least(const Planes& s) {
    uint64_t hit;
    if constexpr (RP == 1)
        hit = s.c0 | s.c1 | s.c2;
    else if constexpr (RP == 2)
        hit = s.c1 | s.c2;
    else if constexpr (RP == 3)
        hit = s.c2 | (s.c1 & s.c0);
    else
        hit = s.c2;
    return __popcll(hit);
}

// files with exactly RP-1 holders: those one more holder would tip over the threshold
template <int RP> __device__ __forceinline__ uint64_t one_short(const Planes& s) {
    if constexpr (RP == 1)
        return ~(s.c0 | s.c1 | s.c2);  // bits above the last file never meet a worker mask
    else if constexpr (RP == 2)
        return s.c0 & ~s.c1 & ~s.c2;
    else if constexpr (RP == 3)
        return s.c1 & ~s.c0 & ~s.c2;
    else
        return s.c0 & s.c1 & ~s.c2;
}

// files with exactly RP-2 holders: those two more holders would tip over the threshold
template <int RP> __device__ __forceinline__ uint64_t two_short(const Planes& s) {
    if constexpr (RP == 1)
        return 0;
    else
        return one_short<RP - 1>(s);
}

struct Best {
    int cnt;
    uint64_t mem;
};

__device__ __forceinline__ void offer(Best& b, int cnt, uint64_t mem) {
    if (cnt > b.cnt || (cnt == b.cnt && mem > b.mem)) {
        b.cnt = cnt;
        b.mem = mem;
    }
}

struct WcResult {
    int32_t count;
    uint32_t pad;
    uint64_t members;
};

// Largest (count, members) of the block -> results[blockIdx.x].  s_cnt / s_mem: kWcBlock entries each.
__device__ __forceinline__ void block_best(const Best& best, int32_t* s_cnt, uint64_t* s_mem,
                                           WcResult* __restrict__ results) {
    s_cnt[threadIdx.x] = best.cnt;
    s_mem[threadIdx.x] = best.mem;
    __syncthreads();
    for (int off = kWcBlock / 2; off > 0; off >>= 1) {
        if (threadIdx.x < off) {
            const int c2 = s_cnt[threadIdx.x + off];
            const uint64_t m2 = s_mem[threadIdx.x + off];
            if (c2 > s_cnt[threadIdx.x] || (c2 == s_cnt[threadIdx.x] && m2 > s_mem[threadIdx.x])) {
                s_cnt[threadIdx.x] = c2;
                s_mem[threadIdx.x] = m2;
            }
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        results[blockIdx.x].count = s_cnt[0];
        results[blockIdx.x].pad = 0;
        results[blockIdx.x].members = s_mem[0];
    }
}

// Copies the per-block results back, waits for the stream and writes the overall maximum
// (worker u sits at bit 63-u of members, so the larger word is the lexicographically earlier set).
inline int collect_best(const WcResult* dev, int blocks, int K, int q, int32_t* c_max, int32_t* argmax, cudaStream_t s) {
    static thread_local WcResult host[kWcMaxBlocks];
    cudaError_t e = cudaMemcpyAsync(host, dev, sizeof(WcResult) * blocks, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_failed(e);
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_failed(e);
    int32_t best_cnt = host[0].count;
    uint64_t best_mem = host[0].members;
    for (int b = 1; b < blocks; ++b)
        if (host[b].count > best_cnt || (host[b].count == best_cnt && host[b].members > best_mem)) {
            best_cnt = host[b].count;
            best_mem = host[b].members;
        }
    if (best_cnt < 0) return BZ_ERR_CUDA;  // no thread saw a subset: cannot happen for a valid launch
    *c_max = best_cnt;
    if (argmax) {
        int t = 0;
        for (int u = 0; u < K && t < q; ++u)
            if (best_mem & (1ull << (63 - u))) argmax[t++] = u;
    }
    return BZ_OK;
}

}  // namespace bz
