// Fused vote + median, staged through shared memory by the TMA unit.
//
// One producer thread per CTA issues cp.async.bulk.tensor loads of boxes
// [R copies][FC files][kTileD coordinates] from a rank-3 tensor map over replicas[r][f][d] into a
// ring of shared-memory stages; four consumer warps take one coordinate per thread, vote the FC
// files of a stage straight out of shared memory and keep the winners' order keys in registers.
// After the last file chunk of a coordinate tile the median network runs and one float is stored.
// The bytes in flight are set by the ring (stages x ~37 KB per CTA), not by registers, and every
// replica byte is read from HBM exactly once.  Every load is a plain per-CTA load of this GPU's own memory.
//
// Every mbarrier wait is bounded: on expiry the kernel raises g_pipeline_timeouts, stops taking
// new tiles, drains the loads it has already issued (bounded as well) and returns.
#include "tma_pipeline.cuh"

#ifndef BZ_VM_MAX_ON_FMA
#define BZ_VM_MAX_ON_FMA 2
#define BZ_VM_MAX_OF 3
#endif

namespace bz {

namespace {

constexpr int kTileD = 128;            // coordinates per tile = consumer threads per CTA
constexpr int kConsumers = kTileD;
constexpr int kThreads = kConsumers + 32;
__device__ unsigned int g_pipeline_timeouts = 0;

template <int R, int F, int FC> struct Shape {
    static constexpr int kChunks = (F + FC - 1) / FC;
    static constexpr int kStageFloats = R * FC * kTileD;
    static constexpr int kStageBytes = kStageFloats * 4;
};

// Dynamic shared memory: [STAGES][R][FC][kTileD] floats (each stage 128-byte aligned), then the
// full/empty barriers.
// VOTE_ONLY: the winners themselves go to out[file * ld_out + j] (bz_vote through the same ring: the loads no
// longer depend on how the rows sit relative to 128-byte lines); otherwise out[j] is their median.
template <int R, int F, int FC, int STAGES, bool VOTE_ONLY = false>
__global__ void __launch_bounds__(kThreads)
    vote_median_tma_kernel(const __grid_constant__ CUtensorMap map, int64_t d, float* __restrict__ out, int64_t ld_out,
                           const ModelUpdate upd) {
    using S = Shape<R, F, FC>;
    // where the ALU pipe limits the kernel (measured), two of three comparators compute their max on the other pipe
    constexpr int kMaxOnFma = (R == 1 || (R == 5 && F == 49)) ? BZ_VM_MAX_ON_FMA : 0, kMaxOf = BZ_VM_MAX_OF;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    float* stages = reinterpret_cast<float*>(smem_raw);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw + static_cast<size_t>(STAGES) * S::kStageBytes);
    uint64_t* empty = full + STAGES;

    const int tid = threadIdx.x;
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kConsumers / 32);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const int64_t n_tiles = (d + kTileD - 1) / kTileD;
    const int64_t my_tiles = blockIdx.x < n_tiles ? (n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    const int64_t n_items = my_tiles * S::kChunks;  // (tile, file chunk) pairs this CTA streams

    if (tid >= kConsumers) {
        // ---------------------------------------------------------------- producer warp
        if (tid == kConsumers) {
            int64_t issued = 0;
            bool alive = true;
            for (; issued < n_items && alive; ++issued) {
                const int s = static_cast<int>(issued % STAGES);
                const uint32_t round = static_cast<uint32_t>(issued / STAGES);
                if (round > 0 && !mbar_wait(&empty[s], (round - 1) & 1)) {
                    alive = false;
                    break;
                }
                const int64_t tile = blockIdx.x + (issued / S::kChunks) * gridDim.x;
                const int chunk = static_cast<int>(issued % S::kChunks);
                mbar_expect_tx(&full[s], S::kStageBytes);
                tma_load_3d(stages + static_cast<size_t>(s) * S::kStageFloats, &map, &full[s],
                            static_cast<int>(tile * kTileD), chunk * FC, 0);
            }
            if (!alive) {
                atomicAdd(&g_pipeline_timeouts, 1u);
                // shared memory must outlive the loads already issued: wait for each stage's last load
                for (int64_t it = issued > STAGES ? issued - STAGES : 0; it < issued; ++it)
                    mbar_wait(&full[it % STAGES], static_cast<uint32_t>(it / STAGES) & 1);
            }
        }
    } else {
        // ---------------------------------------------------------------- consumers: one coordinate each
        int key[VOTE_ONLY ? 1 : F];
        // vote only: 128-bit stores where the output allows them (16-byte aligned rows, whole groups of four)
        const bool wide_out = VOTE_ONLY && ((reinterpret_cast<uintptr_t>(out) | static_cast<uintptr_t>(ld_out * 4)) & 15) == 0 && (d & 3) == 0;
        const bool has_w = upd.w != nullptr, has_v = upd.v != nullptr;
        int64_t item = 0;
        bool alive = true;
        for (int64_t t = 0; t < my_tiles && alive; ++t) {
            const int64_t j = (blockIdx.x + t * gridDim.x) * kTileD + tid;
            // the state this coordinate's update needs is requested now, so that its latency is spent
            // under the votes and the median network rather than after them
            float w_old = 0.f, v_old = 0.f;
            if (has_w && j < d) {
                w_old = upd.w[j];
                if (has_v) v_old = upd.v[j];
            }
#pragma unroll
            for (int chunk = 0; chunk < S::kChunks; ++chunk, ++item) {
                const int s = static_cast<int>(item % STAGES);
                if (!mbar_wait(&full[s], static_cast<uint32_t>(item / STAGES) & 1)) {
                    alive = false;
                    break;
                }
                const uint32_t* base = reinterpret_cast<const uint32_t*>(stages + static_cast<size_t>(s) * S::kStageFloats) + tid;
#pragma unroll
                for (int fi = 0; fi < FC; ++fi) {
                    if (chunk * FC + fi < F) {
                        uint32_t copies[R];
#pragma unroll
                        for (int k = 0; k < R; ++k) copies[k] = base[(k * FC + fi) * kTileD];
                        if constexpr (VOTE_ONLY) {
                            // the winner takes copy 0's place in the stage (only this thread reads that column)
                            if (wide_out)
                                const_cast<uint32_t*>(base)[fi * kTileD] = vote_bits<R>(copies);
                            else if (j < d)
                                out[(chunk * FC + fi) * ld_out + j] = __uint_as_float(vote_bits<R>(copies));
                        } else {
                            key[chunk * FC + fi] = order_key(vote_bits<R>(copies));
                        }
                    }
                }
                __syncwarp();
                if constexpr (VOTE_ONLY) {
                    if (wide_out) {
                        // the warp's 32 columns of the FC winner rows leave as 128-bit stores: lane -> (row, four columns)
                        const int warp = tid >> 5, lane = tid & 31;
                        const int64_t j4 = (blockIdx.x + t * gridDim.x) * kTileD + warp * 32;
                        const float* rows = stages + static_cast<size_t>(s) * S::kStageFloats + warp * 32;
                        for (int idx = lane; idx < FC * 8; idx += 32) {
                            const int row = idx >> 3, c4 = (idx & 7) * 4;
                            if (chunk * FC + row < F && j4 + c4 < d) {   // d is a multiple of 4 on this path
                                const float4 w = *reinterpret_cast<const float4*>(rows + row * kTileD + c4);
                                __stcs(reinterpret_cast<float4*>(out + (chunk * FC + row) * ld_out + j4 + c4), w);
                            }
                        }
                        // this thread wrote the stage through the generic proxy; the bulk copy that refills it
                        // writes through the asynchronous one
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                    }
                }
                if ((tid & 31) == 0) mbar_arrive(&empty[s]);  // this warp is done reading the stage
            }
            if constexpr (!VOTE_ONLY) {
                if (alive && j < d) {
                    const float med = __uint_as_float(key_bits(MedianNet<F>::template run<kMaxOnFma, kMaxOf>(key)));
                    if (out != nullptr) out[j] = med;
                    if (has_w) {
                        upd.w[j] = update_lane(w_old, v_old, med, upd.eta, upd.mu, has_v);
                        if (has_v) upd.v[j] = v_old;
                    }
                }
            }
        }
        if (!alive && (tid & 31) == 0) atomicAdd(&g_pipeline_timeouts, 1u);
    }
}

// ---- host side ----------------------------------------------------------------------------------

template <int R, int F, int FC, int STAGES, bool VOTE_ONLY = false>
int launch_tma(const float* rep, int64_t d, int64_t ld_file, int64_t ld_rep, float* out, int64_t ld_out, const ModelUpdate& upd,
               cudaStream_t s) {
    using S = Shape<R, F, FC>;
    EncodeTiledFn enc = encode_tiled();
    if (enc == nullptr) return 1;
    CUtensorMap map;
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(F), static_cast<cuuint64_t>(R)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(ld_file) * 4, static_cast<cuuint64_t>(R > 1 ? ld_rep : ld_file * F) * 4};
    const cuuint32_t box[3] = {kTileD, FC, R};
    const cuuint32_t elem[3] = {1, 1, 1};
    const CUresult cr = enc(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(rep), dims, strides, box, elem,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return 1;  // shape the descriptor cannot express: use the register path
    constexpr int smem = STAGES * S::kStageBytes + 2 * STAGES * 8;
    auto kern = vote_median_tma_kernel<R, F, FC, STAGES, VOTE_ONLY>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return cuda_failed(e);
    constexpr int fit = (227 * 1024) / (smem + 1024);  // CTAs whose rings fit in one SM (1 KB reserved each)
    constexpr int ctas_per_sm = fit >= 4 ? 4 : (fit >= 1 ? fit : 1);
    int64_t grid = (d + kTileD - 1) / kTileD;
    if (grid > kNumSMs * ctas_per_sm) grid = kNumSMs * ctas_per_sm;
    kern<<<static_cast<int>(grid), kThreads, smem, s>>>(map, d, out, ld_out, upd);
    note_launch();
    return check_launch();
}

}  // namespace

// Returns BZ_OK / an error, or 1 when this path does not apply and the caller should use the
// register path.  Requirements: 16-byte aligned base, leading dimensions multiples of 4 floats,
// d below 2^31, a specialised (r, f).
int vote_median_tma(const float* rep, int r, int f, int64_t d, int64_t ld_file, int64_t ld_rep, float* out,
                    const ModelUpdate& upd, cudaStream_t s) {
    if (!aligned16(rep) || (ld_file % 4) != 0 || (r > 1 && (ld_rep % 4) != 0) || d >= (int64_t(1) << 31)) return 1;
    if (d < 4 * kTileD) return 1;  // tiny inputs: not worth a descriptor
#define BZ_TMA_CASE(R_, F_, FC_, ST_) \
    if (r == R_ && f == F_) return launch_tma<R_, F_, FC_, ST_>(rep, d, ld_file, ld_rep, out, 0, upd, s);
    BZ_TMA_CASE(3, 25, 25, 3)
    BZ_TMA_CASE(3, 49, 25, 3)
    BZ_TMA_CASE(5, 25, 13, 2)
    BZ_TMA_CASE(5, 49, 13, 2)
    BZ_TMA_CASE(7, 49, 10, 2)
    BZ_TMA_CASE(1, 25, 25, 4)
    BZ_TMA_CASE(1, 49, 49, 2)
#undef BZ_TMA_CASE
    return 1;
}

// bz_vote through the ring.  Returns BZ_OK / an error, or 1 when this path does not apply (same requirements as
// above, and ld_voted a multiple of 4 is not needed: the winners are stored with 32-bit stores, one line per warp).
int vote_tma(const float* rep, int r, int f, int64_t d, int64_t ld_file, int64_t ld_rep, float* voted, int64_t ld_voted,
             cudaStream_t s) {
    if (!aligned16(rep) || (ld_file % 4) != 0 || (ld_rep % 4) != 0 || d >= (int64_t(1) << 31) || d < 4 * kTileD) return 1;
    const ModelUpdate none{nullptr, nullptr, 0.f, 0.f};
#define BZ_TMA_VOTE(R_, F_, FC_, ST_) \
    if (r == R_ && f == F_) return launch_tma<R_, F_, FC_, ST_, true>(rep, d, ld_file, ld_rep, voted, ld_voted, none, s);
    BZ_TMA_VOTE(3, 25, 25, 3)
    BZ_TMA_VOTE(3, 49, 25, 3)
    BZ_TMA_VOTE(5, 25, 13, 2)
    BZ_TMA_VOTE(5, 49, 13, 2)
    BZ_TMA_VOTE(7, 49, 10, 2)
#undef BZ_TMA_VOTE
    return 1;
}

int pipeline_timeouts(unsigned int* count) {
    const cudaError_t e = cudaMemcpyFromSymbol(count, g_pipeline_timeouts, sizeof(unsigned int));
    return e == cudaSuccess ? BZ_OK : cuda_failed(e);
}

}  // namespace bz
