// Register tiling of the pairwise-distance kernels: which thread owns which row pairs, the inner
// product-of-differences loop over one shared-memory tile, and the final reduction over CTAs.
#pragma once

#include "bz_common.cuh"

namespace bz {

// The F rows are split into NB = F/T residue classes; a thread owns one unordered pair of classes
// (bi <= bj), i.e. the T x T row pairs (bi + NB*t, bj + NB*u), and one of G interleaved coordinate
// groups of every tile.
template <int F, int T, int G> struct PairTile {
    static constexpr int NB = F / T;
    static constexpr int NPB = NB * (NB + 1) / 2;
    static constexpr int NT = NPB * G;
    static constexpr int TT = T * T;
    static_assert(NB * T == F, "T must divide F");
};

constexpr int kTD = 128;        // coordinates per tile
constexpr int kRowPad = 4;      // floats; keeps the row stride an odd number of 16-byte units
constexpr int kRowStride = kTD + kRowPad;
constexpr int kFlush = 8;       // tiles between two flushes of the binary32 accumulators

// shared memory of the unfused kernel: two stages, the flush buffer, the binary64 sums
template <int F, int T, int G> constexpr size_t tiled_smem_bytes() {
    using PT = PairTile<F, T, G>;
    return size_t(2) * F * kRowStride * 4 + (size_t(PT::NT) * PT::TT + 1) * 4 + size_t(PT::NPB) * PT::TT * 8;
}

// CTAs per SM the launch asks for: as many as the shared memory holds (1 KB reserved each), at most 3.
// Two or more let one CTA's barrier waits overlap another CTA's arithmetic.
template <int F, int T, int G> constexpr int tiled_ctas_per_sm() {
    const int fit = static_cast<int>((227 * 1024) / (tiled_smem_bytes<F, T, G>() + 1024));
    return fit >= 3 ? 3 : (fit >= 1 ? fit : 1);
}

// thread index -> (bi, bj, g)
template <int F, int T, int G> __device__ __forceinline__ void pair_of_thread(int tid, int& bi, int& bj, int& g) {
    using PT = PairTile<F, T, G>;
    const int pb = tid % PT::NPB;
    g = tid / PT::NPB;
    bi = 0;
    int rest = pb;
    while (rest >= PT::NB - bi) {
        rest -= PT::NB - bi;
        ++bi;
    }
    bj = bi + rest;
}

// acc[t*T + u] += sum over this thread's coordinates of the tile of (row(bi,t) - row(bj,u))^2.
// base: [F][kRowStride] floats in shared memory.
template <int F, int T, int G>
__device__ __forceinline__ void accumulate_tile(const float* base, int bi, int bj, int g, float (&acc)[T * T]) {
    constexpr int NB = PairTile<F, T, G>::NB;
#pragma unroll 1
    for (int c4 = g; c4 < kTD / 4; c4 += G) {
        float4 b[T];
#pragma unroll
        for (int u = 0; u < T; ++u) b[u] = *reinterpret_cast<const float4*>(base + (bj + NB * u) * kRowStride + 4 * c4);
#pragma unroll
        for (int t = 0; t < T; ++t) {
            const float4 a = *reinterpret_cast<const float4*>(base + (bi + NB * t) * kRowStride + 4 * c4);
#pragma unroll
            for (int u = 0; u < T; ++u) {
                float s = acc[t * T + u];
                float e;
                e = a.x - b[u].x; s = fmaf(e, e, s);
                e = a.y - b[u].y; s = fmaf(e, e, s);
                e = a.z - b[u].z; s = fmaf(e, e, s);
                e = a.w - b[u].w; s = fmaf(e, e, s);
                acc[t * T + u] = s;
            }
        }
    }
}

// dist[a][b] = sum over CTAs (ascending) of the element of the pair's class block
template <int F, int T, int G>
__global__ void pairdist_tiled_reduce_kernel(const double* __restrict__ partial, int n_ctas, double* __restrict__ dist,
                                             const int* __restrict__ gate = nullptr) {
    using PT = PairTile<F, T, G>;
    if (gate != nullptr && *gate == 0) return;  // nothing was summed: the distances already there stand
    constexpr int NB = PT::NB, NPB = PT::NPB, TT = PT::TT;
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= F * F) return;
    const int a = p / F, b = p % F;
    if (a > b) return;
    if (a == b) {
        dist[p] = 0.0;
        return;
    }
    const int ra = a % NB, ta = a / NB, rb = b % NB, tb = b / NB;
    int bi, bj, t, u;
    if (ra <= rb) {
        bi = ra; bj = rb; t = ta; u = tb;
    } else {
        bi = rb; bj = ra; t = tb; u = ta;
    }
    // index of (bi, bj) among the pairs bi <= bj in row-major order
    const int pb = bi * NB - bi * (bi - 1) / 2 + (bj - bi);
    double s = 0.0;
    for (int cta = 0; cta < n_ctas; ++cta) s += partial[(static_cast<size_t>(cta) * NPB + pb) * TT + t * T + u];
    dist[a * F + b] = s;
    dist[b * F + a] = s;
}

// specialisations: <F, T, G>
#define BZ_PD_25 25, 5, 16
#define BZ_PD_49 49, 7, 8

}  // namespace bz
