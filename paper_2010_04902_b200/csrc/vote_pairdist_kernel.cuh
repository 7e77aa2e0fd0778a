// The kernel of the single-pass vote + pairwise distances.  Included by vote_pairdist.cu only.
//
// A producer thread streams boxes [R copies][FC files][kTD coordinates] of a rank-3 tensor map over
// replicas[r][f][d] into a ring of stages (cp.async.bulk.tensor, plain per-CTA loads, one mbarrier pair
// per stage).  All other warps do both jobs, tile after tile:
//   vote     box by box, every thread takes one 16-byte slot (file, column group): it reads the R
//            copies from the ring, votes them and writes the winner to the CTA's [F][kTD] tile in
//            shared memory and to `voted`; each warp hands the box back as soon as it is through;
//   distance after a barrier the same threads run the register-tiled product-of-differences loop of
//            the unfused kernel on the tile; a second barrier frees the tile for the next vote.
// Two or three CTAs share an SM, so one CTA's voting and barrier waits hide under the others'
// arithmetic.
//
// Every mbarrier wait is bounded.  A thread whose wait ran out stops waiting but keeps arriving, the
// warps agree on the failure at the tile's barrier and leave together; the producer waits (bounded)
// for the loads it has issued before it returns.  The failure is counted.
#pragma once

#include "pairdist_tile.cuh"
#include "tma_pipeline.cuh"

namespace bz {

namespace {

__device__ unsigned int g_fused_timeouts = 0;

constexpr int kFlushParts = 4;  // the flush buffer holds a quarter of the sums at a time

template <int R, int F, int T, int G, int FC, int STAGES> struct Fused {
    using PT = PairTile<F, T, G>;
    static constexpr int NT = PT::NT;                    // threads that own row pairs
    static constexpr int NTP = (NT + 31) / 32 * 32;      // voting / distance threads (whole warps)
    static constexpr int kThreads = NTP + 32;            // + the producer's warp
    static constexpr int kChunks = F / FC;
    static constexpr int kStageFloats = R * FC * kTD;
    static constexpr int kStageBytes = kStageFloats * 4;
    static constexpr int kPart = (PT::TT + kFlushParts - 1) / kFlushParts;  // sums per thread in one flush part
    static constexpr int kRedFloats = (NT * kPart + 1) / 2 * 2;
    static constexpr int kTileFloats = F * kRowStride;
    static constexpr size_t kSmem = size_t(STAGES) * kStageBytes + size_t(kTileFloats) * 4 + size_t(kRedFloats) * 4 +
                                    size_t(PT::NPB) * PT::TT * 8 + 2 * STAGES * 8;
    // CTAs per SM: as many as the shared memory holds (1 KB reserved each), at most 3; while one CTA
    // votes (latency-bound) or waits at a barrier, the others keep the FP32 pipe busy
    static constexpr int kFit = static_cast<int>((227 * 1024) / (kSmem + 1024));
    static constexpr int kCtasPerSm = kFit >= 3 ? 3 : (kFit >= 1 ? kFit : 1);
    static_assert(kSmem + 1024 <= 227 * 1024, "ring, tile and sums must fit one SM");
    static_assert(kChunks * FC == F, "FC must divide F");
    static_assert(kStageBytes % 128 == 0, "stages stay 128-byte aligned");
    static_assert((kTileFloats * 4) % 16 == 0, "tiles stay 16-byte aligned");
};

// barrier 1: the voting / distance threads only
template <int COUNT> __device__ __forceinline__ void compute_sync() { asm volatile("bar.sync 1, %0;" ::"n"(COUNT) : "memory"); }
template <int COUNT> __device__ __forceinline__ bool compute_any(bool flag) {
    uint32_t out;
    asm volatile(
        "{\n"
        ".reg .pred p, q;\n"
        "setp.ne.u32 q, %1, 0;\n"
        "bar.red.or.pred p, 1, %2, q;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(out)
        : "r"(static_cast<uint32_t>(flag)), "n"(COUNT)
        : "memory");
    return out != 0;
}

template <int R, int F, int T, int G, int FC, int STAGES>
__global__ void __launch_bounds__(Fused<R, F, T, G, FC, STAGES>::kThreads, Fused<R, F, T, G, FC, STAGES>::kCtasPerSm)
    vote_pairdist_kernel(const __grid_constant__ CUtensorMap map, int64_t d, float* __restrict__ voted, int64_t ld_voted,
                         double* __restrict__ partial) {
    using S = Fused<R, F, T, G, FC, STAGES>;
    using PT = typename S::PT;
    constexpr int NPB = PT::NPB, NT = PT::NT, TT = PT::TT, NTP = S::NTP;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    float* stages = reinterpret_cast<float*>(smem_raw);
    float* tile = stages + STAGES * S::kStageFloats;                 // [F][kRowStride] voted values
    float* red = tile + S::kTileFloats;                              // [G][NPB][kPart]
    double* dsum = reinterpret_cast<double*>(red + S::kRedFloats);   // [NPB][TT]
    uint64_t* full = reinterpret_cast<uint64_t*>(dsum + NPB * TT);
    uint64_t* empty = full + STAGES;

    const int tid = threadIdx.x;
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], NTP / 32);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int e = tid; e < NPB * TT; e += S::kThreads) dsum[e] = 0.0;
    __syncthreads();

    const int64_t n_tiles = (d + kTD - 1) / kTD;
    const int64_t my_tiles = blockIdx.x < n_tiles ? (n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    const int64_t n_items = my_tiles * S::kChunks;  // (tile, file chunk) boxes of this CTA

    if (tid >= NTP) {
        // ------------------------------------------------------------------ producer
        if (tid == NTP) {
            int64_t issued = 0;
            bool alive = true;
            for (; issued < n_items; ++issued) {
                const int s = static_cast<int>(issued % STAGES);
                const uint32_t round = static_cast<uint32_t>(issued / STAGES);
                if (round > 0 && !mbar_wait(&empty[s], (round - 1) & 1)) {
                    alive = false;
                    break;
                }
                const int64_t tile_i = blockIdx.x + (issued / S::kChunks) * gridDim.x;
                mbar_expect_tx(&full[s], S::kStageBytes);
                tma_load_3d(stages + static_cast<size_t>(s) * S::kStageFloats, &map, &full[s], static_cast<int>(tile_i * kTD),
                            static_cast<int>(issued % S::kChunks) * FC, 0);
            }
            if (!alive) {
                atomicAdd(&g_fused_timeouts, 1u);
                // shared memory must outlive the loads already issued: wait for each stage's last load
                for (int64_t it = issued > STAGES ? issued - STAGES : 0; it < issued; ++it)
                    mbar_wait(&full[it % STAGES], static_cast<uint32_t>(it / STAGES) & 1);
            }
        }
        return;
    }

    // ---------------------------------------------------------------------- voting / distance warps
    const bool owner = tid < NT;  // the padding threads of the last warp vote but own no row pairs
    int bi = 0, bj = 0, g = 0;
    if (owner) pair_of_thread<F, T, G>(tid, bi, bj, g);
    const int pb = tid % NPB;
    float acc[TT];
#pragma unroll
    for (int e = 0; e < TT; ++e) acc[e] = 0.f;

    int since_flush = 0;
    bool failed = false;
    for (int64_t t = 0; t < my_tiles; ++t) {
        const int64_t item0 = t * S::kChunks;
        const int64_t j0 = (blockIdx.x + t * gridDim.x) * kTD;
        // vote: box by box, every thread one 16-byte slot (file fi, column group c4) of the box
        for (int chunk = 0; chunk < S::kChunks; ++chunk) {
            const int64_t it = item0 + chunk;
            const int s = static_cast<int>(it % STAGES);
            if (!failed && !mbar_wait(&full[s], static_cast<uint32_t>(it / STAGES) & 1)) failed = true;
            if (!failed) {
                const float* box = stages + static_cast<size_t>(s) * S::kStageFloats;
                for (int slot = tid; slot < FC * (kTD / 4); slot += NTP) {
                    const int fi = slot / (kTD / 4), c4 = slot - fi * (kTD / 4);
                    uint4 x[R];
#pragma unroll
                    for (int k = 0; k < R; ++k) x[k] = *reinterpret_cast<const uint4*>(box + (k * FC + fi) * kTD + 4 * c4);
                    uint32_t c0[R], c1[R], c2[R], c3[R];
#pragma unroll
                    for (int k = 0; k < R; ++k) {
                        c0[k] = x[k].x;
                        c1[k] = x[k].y;
                        c2[k] = x[k].z;
                        c3[k] = x[k].w;
                    }
                    const uint4 w = make_uint4(vote_bits<R>(c0), vote_bits<R>(c1), vote_bits<R>(c2), vote_bits<R>(c3));
                    const int row = chunk * FC + fi;
                    *reinterpret_cast<uint4*>(tile + row * kRowStride + 4 * c4) = w;  // columns past d hold the fill value 0
                    const int64_t j = j0 + 4 * c4;
                    float* dst = voted + row * ld_voted + j;
                    if (j + 3 < d) {
                        *reinterpret_cast<uint4*>(dst) = w;
                    } else {
                        if (j < d) dst[0] = __uint_as_float(w.x);
                        if (j + 1 < d) dst[1] = __uint_as_float(w.y);
                        if (j + 2 < d) dst[2] = __uint_as_float(w.z);
                    }
                }
            }
            __syncwarp();
            if ((tid & 31) == 0) mbar_arrive(&empty[s]);  // this warp is done with the box (or has given up on it)
        }
        if (compute_any<NTP>(failed)) {  // also publishes the tile to every warp
            failed = true;
            break;
        }
        if (owner) accumulate_tile<F, T, G>(tile, bi, bj, g, acc);
        ++since_flush;
        if (since_flush == kFlush || t + 1 == my_tiles) {  // uniform over the CTA
            since_flush = 0;
#pragma unroll
            for (int part = 0; part < kFlushParts; ++part) {
                constexpr int P = S::kPart;
                if (owner) {
#pragma unroll
                    for (int i = 0; i < P; ++i)
                        if (part * P + i < TT) {
                            red[tid * P + i] = acc[part * P + i];  // tid = g * NPB + pb
                            acc[part * P + i] = 0.f;
                        }
                }
                compute_sync<NTP>();
                if (owner)
                    for (int i = g; i < P && part * P + i < TT; i += G) {
                        float sum = 0.f;
#pragma unroll
                        for (int g2 = 0; g2 < G; ++g2) sum += red[(g2 * NPB + pb) * P + i];
                        dsum[pb * TT + part * P + i] += static_cast<double>(sum);
                    }
                compute_sync<NTP>();  // the buffer may be refilled
            }
        } else {
            compute_sync<NTP>();  // every warp is done with the tile: it may be voted over
        }
    }
    if (failed && (tid & 31) == 0) atomicAdd(&g_fused_timeouts, 1u);
    double* mine = partial + static_cast<size_t>(blockIdx.x) * NPB * TT;
    for (int e = tid; e < NPB * TT; e += NTP) mine[e] = dsum[e];
}

}  // namespace

}  // namespace bz
