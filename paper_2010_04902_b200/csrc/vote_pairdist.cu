// Majority vote (Eq. 3) and the pairwise distances of the Krum family (Sec. 1.2) in one pass over the
// replicas: the winners are written to `voted` and go straight from shared memory into the distance
// sums, so the f voted rows are not read back from HBM (4*f bytes per coordinate saved).
//
// The kernel (vote_pairdist_kernel.cuh) streams the replicas through a TMA ring, votes them into
// tiles of shared memory and runs the distance arithmetic of the unfused kernel on those tiles.
// Partial sums and their reduction are those of the unfused kernel.
#include "vote_pairdist_kernel.cuh"

namespace bz {

int pairdist_on_device(const float* v, int f, int64_t d, int64_t ld, double* dist, void* ws, cudaStream_t s, bool tensor_cores);  // pairdist.cu
size_t pairdist_workspace(int f);
size_t pairdist_workspace_fp32(int f);
int pairdist_fp32(const float* v, int f, int64_t d, int64_t ld, double* dist, double* partial, const int* gate, cudaStream_t s);
int pairdist_f64(const float* v, int f, int64_t d, int64_t ld, double* dist, double* partial, const int* gate, cudaStream_t s);
int pairdist_path_fp32_only();
int pairdist_path_fp64_only();
int pairdist_path_i8_forced();
int vote_pairdist_i8(const float* rep, int r, int f, int64_t d, int64_t ld_file, int64_t ld_rep, float* voted, int64_t ld_voted,
                     double* dist, void* ws, int* flag, int force, cudaStream_t s);  // pairdist_i8.cu
int* pairdist_status_words(void* ws, int f);   // pairdist.cu
void* pairdist_i8_part(void* ws, int f);
int pairdist_clear_status(void* ws, int f, cudaStream_t s);
int vote_if(const float* replicas, int r, int f, int64_t d, int64_t ld_file, int64_t ld_replica, float* voted,
            int64_t ld_voted, const int* gate, cudaStream_t s);  // vote_median.cu
size_t krum_workspace_bytes(int op, int f);
int check_workspace(void* ws, size_t have, size_t need);

namespace {

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
    // (r, f, T, G, files per box, ring depth)
    BZ_FUSED_CASE(3, 25, 5, 16, 5, 6)
    BZ_FUSED_CASE(3, 49, 7, 8, 7, 6)
    BZ_FUSED_CASE(5, 25, 5, 16, 5, 4)
    BZ_FUSED_CASE(5, 49, 7, 8, 7, 3)
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
    // Vote + integer distances on the tensor cores wherever that kernel exists (it is the faster single
    // pass on every shape measured).  Two repairs follow, both decided on the device from the kernel's flag
    // words and both returning at once in the ordinary case: the vote alone if the kernel stopped early (its
    // voted rows are then incomplete), and the binary64 distance kernel if it stopped early or its error
    // bound asks for it.
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (d > 0 && r > 1 && !pairdist_path_fp32_only() && !pairdist_path_fp64_only()) {
        int* flag = pairdist_status_words(workspace, f);
        st = vote_pairdist_i8(replicas, r, f, d, ld_file, ld_replica, voted, ld_voted, dist, pairdist_i8_part(workspace, f), flag,
                              pairdist_path_i8_forced(), s);
        if (st == BZ_OK) {
            note_path(BZ_PATH_TENSOR);
            st = vote_if(replicas, r, f, d, ld_file, ld_replica, voted, ld_voted, flag + 1, s);
            if (st != BZ_OK) return st;
            return pairdist_f64(voted, f, d, ld_voted, dist, static_cast<double*>(workspace), flag, s);
        }
        if (st != 1) return st;
    }
    // the binary32 single pass: only where the caller asked for binary32 (otherwise the two calls below keep the
    // tolerance on short rows through the binary64 kernel)
    if (d > 0 && r > 1 && pairdist_path_fp32_only()) {
        st = vote_pairdist_fused(replicas, r, f, d, ld_file, ld_replica, voted, ld_voted, dist,
                                 static_cast<double*>(workspace), s);
        if (st == BZ_OK) {
            note_path(BZ_PATH_FP32_FUSED);
            return pairdist_clear_status(workspace, f, s);
        }
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
