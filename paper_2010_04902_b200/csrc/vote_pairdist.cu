// Majority vote (Eq. 3) and the pairwise distances of the Krum family (Sec. 1.2) in one pass over the
// replicas: the winners are written to `voted` and go straight from shared memory into the distance
// sums, so the f voted rows are not read back from HBM (4*f bytes per coordinate saved).
//
// A producer thread streams boxes [R copies][FC files][kTD coordinates] of a rank-3 tensor map over
// replicas[r][f][d] into a ring of stages (cp.async.bulk.tensor, one mbarrier pair per stage; no
// cluster multicast).  The consumer threads vote each box 16 bytes at a time into the CTA's
// [F][kTD] tile - and into `voted` - and, once a tile is complete, run the same register-tiled
// product-of-differences loop as the unfused kernel on it.  Partial sums and their reduction are
// those of the unfused kernel, so the summation order inside a CTA is the same.
//
// Every mbarrier wait is bounded.  A consumer whose wait ran out stops waiting but keeps arriving,
// the consumers agree on the failure at their next common barrier and leave together; the producer
// waits (bounded) for the loads it has issued before it returns.  The failure is counted.
#include "pairdist_tile.cuh"
#include "tma_pipeline.cuh"

namespace bz {

int pairdist_on_device(const float* v, int f, int64_t d, int64_t ld, double* dist, void* ws, cudaStream_t s);  // pairdist.cu
size_t pairdist_workspace(int f);
size_t krum_workspace_bytes(int op, int f);
int check_workspace(void* ws, size_t have, size_t need);

namespace {

__device__ unsigned int g_fused_timeouts = 0;

template <int R, int F, int T, int G, int FC, int STAGES> struct Fused {
    using PT = PairTile<F, T, G>;
    static constexpr int NT = PT::NT;                    // threads that own row pairs
    static constexpr int NTP = (NT + 31) / 32 * 32;      // consumer threads (whole warps)
    static constexpr int kThreads = NTP + 32;            // + the producer's warp
    static constexpr int kChunks = F / FC;
    static constexpr int kStageFloats = R * FC * kTD;
    static constexpr int kStageBytes = kStageFloats * 4;
    static constexpr int kRedFloats = (NT * PT::TT + 1) / 2 * 2;
    static constexpr size_t kSmem = size_t(STAGES) * kStageBytes + size_t(F) * kRowStride * 4 + size_t(kRedFloats) * 4 +
                                    size_t(PT::NPB) * PT::TT * 8 + 2 * STAGES * 8;
    static constexpr int kFit = static_cast<int>((227 * 1024) / (kSmem + 1024));
    static constexpr int kCtasPerSm = kFit >= 3 ? 3 : (kFit >= 1 ? kFit : 1);
    static_assert(kChunks * FC == F, "FC must divide F");
    static_assert(kStageBytes % 128 == 0, "stages stay 128-byte aligned");
};

// barrier 1: the consumer threads only
template <int COUNT> __device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(COUNT) : "memory"); }
template <int COUNT> __device__ __forceinline__ bool consumer_any(bool flag) {
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
    float* tile = stages + STAGES * S::kStageFloats;               // [F][kRowStride] voted values
    float* red = tile + F * kRowStride;                            // [G][NPB][TT]
    double* dsum = reinterpret_cast<double*>(red + S::kRedFloats);  // [NPB][TT]
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
    const int64_t n_items = my_tiles * S::kChunks;

    if (tid >= NTP) {
        // ---------------------------------------------------------------- producer
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
                const int chunk = static_cast<int>(issued % S::kChunks);
                mbar_expect_tx(&full[s], S::kStageBytes);
                tma_load_3d(stages + static_cast<size_t>(s) * S::kStageFloats, &map, &full[s], static_cast<int>(tile_i * kTD),
                            chunk * FC, 0);
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

    // -------------------------------------------------------------------- consumers
    const bool owner = tid < NT;  // the padding threads of the last warp only keep the barriers whole
    int bi = 0, bj = 0, g = 0;
    if (owner) pair_of_thread<F, T, G>(tid, bi, bj, g);
    const int pb = tid % NPB;
    float acc[TT];
#pragma unroll
    for (int e = 0; e < TT; ++e) acc[e] = 0.f;

    int64_t item = 0;
    int since_flush = 0;
    bool failed = false;
    for (int64_t t = 0; t < my_tiles; ++t) {
        const int64_t j0 = (blockIdx.x + t * gridDim.x) * kTD;
        for (int chunk = 0; chunk < S::kChunks; ++chunk, ++item) {
            const int s = static_cast<int>(item % STAGES);
            if (!failed && !mbar_wait(&full[s], static_cast<uint32_t>(item / STAGES) & 1)) failed = true;
            if (!failed) {
                const float* box = stages + static_cast<size_t>(s) * S::kStageFloats;
                for (int slot = tid; slot < FC * (kTD / 4); slot += NTP) {
                    const int fi = slot / (kTD / 4), c4 = slot - fi * (kTD / 4);
                    uint4 x[R];
#pragma unroll
                    for (int k = 0; k < R; ++k) x[k] = *reinterpret_cast<const uint4*>(box + (k * FC + fi) * kTD + 4 * c4);
                    uint4 w;
                    {
                        uint32_t c0[R], c1[R], c2[R], c3[R];
#pragma unroll
                        for (int k = 0; k < R; ++k) {
                            c0[k] = x[k].x;
                            c1[k] = x[k].y;
                            c2[k] = x[k].z;
                            c3[k] = x[k].w;
                        }
                        w = make_uint4(vote_bits<R>(c0), vote_bits<R>(c1), vote_bits<R>(c2), vote_bits<R>(c3));
                    }
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
            if ((tid & 31) == 0) mbar_arrive(&empty[s]);  // this warp is done with the stage (or has given up on it)
        }
        if (consumer_any<NTP>(failed)) {  // also publishes the tile to every consumer
            failed = true;
            break;
        }
        if (owner) accumulate_tile<F, T, G>(tile, bi, bj, g, acc);
        ++since_flush;
        if (since_flush == kFlush || t + 1 == my_tiles) {  // uniform over the CTA
            since_flush = 0;
            if (owner) {
#pragma unroll
                for (int e = 0; e < TT; ++e) {
                    red[tid * TT + e] = acc[e];  // tid = g * NPB + pb
                    acc[e] = 0.f;
                }
            }
            consumer_sync<NTP>();
            if (owner)
                for (int e = g; e < TT; e += G) {
                    float sum = 0.f;
#pragma unroll
                    for (int g2 = 0; g2 < G; ++g2) sum += red[(g2 * NPB + pb) * TT + e];
                    dsum[pb * TT + e] += static_cast<double>(sum);
                }
        }
        consumer_sync<NTP>();  // the tile may be overwritten, the sums are in place
    }
    if (failed && (tid & 31) == 0) atomicAdd(&g_fused_timeouts, 1u);
    double* mine = partial + static_cast<size_t>(blockIdx.x) * NPB * TT;
    for (int e = tid; e < NPB * TT; e += NTP) mine[e] = dsum[e];
}

template <int R, int F, int T, int G, int FC, int STAGES>
int launch_fused(const float* rep, int64_t d, int64_t ld_file, int64_t ld_rep, float* voted, int64_t ld_voted, double* dist,
                 double* partial, cudaStream_t s) {
    using S = Fused<R, F, T, G, FC, STAGES>;
    static_assert(S::kCtasPerSm <= tiled_ctas_per_sm<F, T, G>(), "the partial sums must fit the unfused kernel's workspace");
    EncodeTiledFn enc = encode_tiled();
    if (enc == nullptr) return 1;
    CUtensorMap map;
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(F), static_cast<cuuint64_t>(R)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(ld_file) * 4, static_cast<cuuint64_t>(ld_rep) * 4};
    const cuuint32_t box[3] = {kTD, FC, R};
    const cuuint32_t elem[3] = {1, 1, 1};
    const CUresult cr = enc(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(rep), dims, strides, box, elem,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return 1;
    auto kern = vote_pairdist_kernel<R, F, T, G, FC, STAGES>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(S::kSmem));
    if (e != cudaSuccess) return cuda_failed(e);
    int64_t ctas = (d + kTD - 1) / kTD;
    if (ctas > kNumSMs * S::kCtasPerSm) ctas = kNumSMs * S::kCtasPerSm;
    kern<<<static_cast<int>(ctas), S::kThreads, S::kSmem, s>>>(map, d, voted, ld_voted, partial);
    note_launch();
    int st = check_launch();
    if (st != BZ_OK) return st;
    pairdist_tiled_reduce_kernel<F, T, G><<<(F * F + 127) / 128, 128, 0, s>>>(partial, static_cast<int>(ctas), dist);
    note_launch();
    return check_launch();
}

// BZ_OK / error, or 1 when no fused kernel applies (shape, alignment, size)
int vote_pairdist_fused(const float* rep, int r, int f, int64_t d, int64_t ld_file, int64_t ld_rep, float* voted,
                        int64_t ld_voted, double* dist, double* partial, cudaStream_t s) {
    if (!aligned16(rep) || !aligned16(voted) || (ld_file % 4) != 0 || (ld_rep % 4) != 0 || (ld_voted % 4) != 0) return 1;
    if (d >= (int64_t(1) << 31) || d < 4 * kTD) return 1;
#define BZ_FUSED_CASE(R_, F_, T_, G_, FC_, ST_) \
    if (r == R_ && f == F_) return launch_fused<R_, F_, T_, G_, FC_, ST_>(rep, d, ld_file, ld_rep, voted, ld_voted, dist, partial, s);
    BZ_FUSED_CASE(3, 25, 5, 16, 5, 3)
    BZ_FUSED_CASE(3, 49, 7, 8, 7, 3)
    BZ_FUSED_CASE(5, 25, 5, 16, 5, 3)
    BZ_FUSED_CASE(5, 49, 7, 8, 7, 2)
    BZ_FUSED_CASE(7, 49, 7, 8, 7, 2)
#undef BZ_FUSED_CASE
    return 1;
}

}  // namespace

int vote_pairdist_timeouts(unsigned int* count) {
    const cudaError_t e = cudaMemcpyFromSymbol(count, g_fused_timeouts, sizeof(unsigned int));
    return e == cudaSuccess ? BZ_OK : cuda_failed(e);
}

}  // namespace bz

using namespace bz;

extern "C" int bz_vote_pairdist(const float* replicas, int r, int f, int64_t d, int64_t ld_file, int64_t ld_replica,
                                float* voted, int64_t ld_voted, double* dist, void* workspace, size_t workspace_bytes,
                                void* stream) {
    // the argument rules of bz_vote followed by bz_pairdist
    if (dist == nullptr || d < 0 || r < 1 || f < 1 || (r % 2) == 0) return BZ_ERR_INVALID_ARG;
    if ((replicas == nullptr || voted == nullptr) && d > 0) return BZ_ERR_INVALID_ARG;
    if (r > BZ_MAX_R || f > BZ_MAX_F) return BZ_ERR_UNSUPPORTED;
    if (ld_file < d || (r > 1 && ld_replica < d) || ld_voted < d) return BZ_ERR_INVALID_ARG;
    int st = check_workspace(workspace, workspace_bytes, krum_workspace_bytes(BZ_OP_PAIRDIST, f));
    if (st != BZ_OK) return st;
    if (d > 0 && r > 1) {
        st = vote_pairdist_fused(replicas, r, f, d, ld_file, ld_replica, voted, ld_voted, dist,
                                 static_cast<double*>(workspace), static_cast<cudaStream_t>(stream));
        if (st != 1) return st;
    }
    // shapes without a fused kernel: the two calls this one stands for
    st = bz_vote(replicas, r, f, d, ld_file, ld_replica, voted, ld_voted, stream);
    if (st != BZ_OK) return st;
    return bz_pairdist(voted, f, d, ld_voted, dist, workspace, workspace_bytes, stream);
}

extern "C" int bz_vote_multikrum(const float* replicas, int r, int f, int64_t d, int64_t ld_file, int64_t ld_replica,
                                 int c, int m, float* voted, int64_t ld_voted, float* out, int32_t* selected, double* dist,
                                 void* workspace, size_t workspace_bytes, void* stream) {
    if ((out == nullptr && d > 0) || selected == nullptr) return BZ_ERR_INVALID_ARG;
    if (f < 1 || f > BZ_MAX_F) return f < 1 ? BZ_ERR_INVALID_ARG : BZ_ERR_UNSUPPORTED;
    if (c < 0 || f < 2 * c + 3 || m < 1 || m > f) return BZ_ERR_PRECONDITION;
    int st = check_workspace(workspace, workspace_bytes, krum_workspace_bytes(BZ_OP_MULTIKRUM, f));
    if (st != BZ_OK) return st;
    double* D = dist ? dist : reinterpret_cast<double*>(static_cast<char*>(workspace) + pairdist_workspace(f));
    st = bz_vote_pairdist(replicas, r, f, d, ld_file, ld_replica, voted, ld_voted, D, workspace, pairdist_workspace(f), stream);
    if (st != BZ_OK) return st;
    st = bz_krum_select(D, f, c, m, selected, stream);
    if (st != BZ_OK) return st;
    return bz_mean_rows(voted, f, d, ld_voted, selected, m, out, stream);
}

extern "C" int bz_vote_bulyan(const float* replicas, int r, int f, int64_t d, int64_t ld_file, int64_t ld_replica, int c,
                              float* voted, int64_t ld_voted, float* out, int32_t* selected, void* workspace,
                              size_t workspace_bytes, void* stream) {
    if ((out == nullptr && d > 0) || selected == nullptr) return BZ_ERR_INVALID_ARG;
    if (f < 1 || f > BZ_MAX_F) return f < 1 ? BZ_ERR_INVALID_ARG : BZ_ERR_UNSUPPORTED;
    if (c < 0 || f < 4 * c + 3) return BZ_ERR_PRECONDITION;
    int st = check_workspace(workspace, workspace_bytes, krum_workspace_bytes(BZ_OP_BULYAN, f));
    if (st != BZ_OK) return st;
    double* D = reinterpret_cast<double*>(static_cast<char*>(workspace) + pairdist_workspace(f));
    st = bz_vote_pairdist(replicas, r, f, d, ld_file, ld_replica, voted, ld_voted, D, workspace, pairdist_workspace(f), stream);
    if (st != BZ_OK) return st;
    st = bz_bulyan_select(D, f, c, selected, stream);
    if (st != BZ_OK) return st;
    const int theta = f - 2 * c;
    return bz_trimmed_mean(voted, f, d, ld_voted, selected, theta, theta - 2 * c, out, stream);
}
