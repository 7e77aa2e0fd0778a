// Pairwise squared distances of the Krum family (Sec. 1.2; cost in Appendix A.1) on the tensor cores,
// in exact integer arithmetic.  Host side; the kernel is in pairdist_i8_kernel.cuh.
#include "pairdist_i8_kernel.cuh"

namespace bz {

namespace {

// D from the CTAs' partial matrices, then the error estimate of the conversion (two small kernels).
// flag[0] = 1 asks for the binary32 kernel: the estimate is above the tolerance (ignored with force != 0),
// a row holds values the fixed-point scale cannot carry, or a CTA stopped early.  flag[1] = 1 says the
// latter: a bounded wait ran out, the partial matrices are incomplete and so are the voted rows of the
// kernel with the vote in front.
// Estimate for a pair: each value is rounded to a multiple of its row's step, an unbiased error of
// standard deviation 0.29 step; over d coordinates that moves D by about 2 sqrt(D var) + d var.
constexpr double kRelTol = 5e-9;

// One warp per pair a <= b: lane l takes CTAs l, l+32, ... in order, then the lanes are added in a fixed
// tree.  Identical rows meet identical numbers in the same order and get identical distances.
template <int F>
__global__ void __launch_bounds__(256)
    pairdist_i8_reduce_kernel(const double* __restrict__ tpart, int n_ctas, double* __restrict__ dist) {
    const int pair = blockIdx.x * (blockDim.x / 32) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (pair >= F * F) return;
    const int a = pair / F, b = pair % F;
    if (a > b) return;
    double s = 0.0;
    if (a < b) {
        for (int c = lane; c < n_ctas; c += 32) {
            const double* T = tpart + static_cast<size_t>(c) * F * F;
            s += (T[a * F + a] + T[b * F + b]) - (T[a * F + b] + T[b * F + a]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
    }
    if (lane == 0) {
        dist[a * F + b] = s;
        dist[b * F + a] = s;
    }
}

// The error estimate and the CTAs' marks -> flag[0], flag[1].
template <int F>
__global__ void __launch_bounds__(256)
    pairdist_i8_check_kernel(const double* __restrict__ dist, const int* __restrict__ info, int n_ctas, int64_t d, int force,
                             int* __restrict__ flag) {
    __shared__ int s_emax[F];
    __shared__ int s_bad, s_marks;
    const int tid = threadIdx.x;
    if (tid == 0) s_bad = s_marks = 0;
    if (tid < F) s_emax[tid] = kELo;
    __syncthreads();
    for (int e = tid; e < n_ctas * kInfoStride; e += blockDim.x) {
        const int a = e % kInfoStride;
        if (a < F) atomicMax(&s_emax[a], info[e]);
        if (a == kInfoBad && info[e]) atomicOr(&s_marks, info[e]);
    }
    __syncthreads();
    // 2 sqrt(x) + d x <= tol  <=>  x <= x_max with sqrt(x_max) = (sqrt(1 + d tol) - 1) / d: one square root
    // per thread instead of one per pair
    const double dd = static_cast<double>(d);
    const double y_max = (sqrt(1.0 + dd * kRelTol) - 1.0) / dd;
    const double x_max = y_max * y_max;
    __shared__ double s_min_nz[F], s_zero_step[F];
    if (tid < F) {
        s_min_nz[tid] = 1e300;
        s_zero_step[tid] = 0.0;
    }
    __syncthreads();
    bool bad = false;
    for (int p = tid; p < F * F; p += blockDim.x) {
        const int a = p / F, b = p % F;
        if (a >= b) continue;
        const double step_a = __longlong_as_double(static_cast<long long>(1023 + s_emax[a] - 30) << 52);
        const double step_b = __longlong_as_double(static_cast<long long>(1023 + s_emax[b] - 30) << 52);
        const double var = 0.0841 * (step_a * step_a + step_b * step_b);
        const double v = dist[a * F + b];
        if (v > 0.0) {
            if (var > x_max * v) bad = true;
            atomicMin(reinterpret_cast<unsigned long long*>(&s_min_nz[a]), static_cast<unsigned long long>(__double_as_longlong(v)));
            atomicMin(reinterpret_cast<unsigned long long*>(&s_min_nz[b]), static_cast<unsigned long long>(__double_as_longlong(v)));
        } else if (v == 0.0) {
            const double z = fmax(step_a, step_b);
            atomicMax(reinterpret_cast<unsigned long long*>(&s_zero_step[a]), static_cast<unsigned long long>(__double_as_longlong(z)));
            atomicMax(reinterpret_cast<unsigned long long*>(&s_zero_step[b]), static_cast<unsigned long long>(__double_as_longlong(z)));
        } else {
            bad = true;
        }
    }
    if (bad) atomicOr(&s_bad, 1);
    __syncthreads();
    // rows that convert to the same integers may still differ by less than a step everywhere
    if (tid < F && s_zero_step[tid] > 0.0 && s_min_nz[tid] < 1e300 &&
        dd * s_zero_step[tid] * s_zero_step[tid] > kRelTol * s_min_nz[tid])
        atomicOr(&s_bad, 1);
    __syncthreads();
    if (tid == 0) {
        flag[0] = ((s_bad && !force) || s_marks) ? 1 : 0;
        flag[1] = (s_marks & kBadStopped) ? 1 : 0;
    }
}

// rep: R = 1: rows [f][d] with leading dimension ld_file.  R > 1: replicas[r][f][d].
// Returns 1 if the tensor map cannot express the shape.
template <int F, int W, int R, int FC, int NS, int TS>
int launch_i8(const float* rep, int64_t d, int64_t ld_file, int64_t ld_rep, float* voted, int64_t ld_voted, double* dist,
              double* tpart, int* info, int* flag, int force, cudaStream_t s) {
    using S = I8Shape<F, W, R, FC, NS, TS>;
    EncodeTiledFn enc = encode_tiled();
    if (enc == nullptr) return 1;
    CUtensorMap map;
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(F), static_cast<cuuint64_t>(R)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(ld_file) * 4, static_cast<cuuint64_t>(R > 1 ? ld_rep : ld_file * F) * 4};
    const cuuint32_t box[3] = {kTK, FC, R};
    const cuuint32_t elem[3] = {1, 1, 1};
    const CUresult cr = enc(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(rep), dims, strides, box, elem,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return 1;
    auto kern = pairdist_i8_kernel<F, W, R, FC, NS, TS>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, S::kSmem);
    if (e != cudaSuccess) return cuda_failed(e);
    int64_t ctas = (d + kTK - 1) / kTK;
    if (ctas > kNumSMs) ctas = kNumSMs;
    kern<<<static_cast<int>(ctas), S::kThreads, S::kSmem, s>>>(map, d, voted, ld_voted, tpart, info);
    note_launch();
    int st = check_launch();
    if (st != BZ_OK) return st;
    pairdist_i8_reduce_kernel<F><<<(F * F + 7) / 8, 256, 0, s>>>(tpart, static_cast<int>(ctas), dist);
    note_launch();
    st = check_launch();
    if (st != BZ_OK) return st;
    pairdist_i8_check_kernel<F><<<1, 256, 0, s>>>(dist, info, static_cast<int>(ctas), d, force, flag);
    note_launch();
    return check_launch();
}

size_t tpart_bytes(int f) { return round_up(static_cast<size_t>(kNumSMs) * f * f * sizeof(double), 256); }
size_t info_bytes() { return round_up(static_cast<size_t>(kNumSMs) * kInfoStride * sizeof(int), 256); }

struct Scratch {
    double* tpart;
    int* info;
};
Scratch carve(void* ws, int f) {
    char* p = static_cast<char*>(ws);
    Scratch s;
    s.tpart = reinterpret_cast<double*>(p);
    p += tpart_bytes(f);
    s.info = reinterpret_cast<int*>(p);
    return s;
}

}  // namespace

bool pairdist_i8_has(int f) { return f == 25 || f == 49; }

// bytes of the partial matrices and the per-CTA records
size_t pairdist_i8_workspace(int f) {
    if (!pairdist_i8_has(f)) return 0;
    return tpart_bytes(f) + info_bytes();
}

// Returns BZ_OK / an error, or 1 when this path does not apply (shape, alignment, size).  On BZ_OK
// dist holds the distances, flag[0] (device) is 1 if they must be recomputed in binary32 and flag[1] is 1
// if the kernel stopped early.
int pairdist_i8(const float* v, int f, int64_t d, int64_t ld, double* dist, void* ws, int* flag, int force, cudaStream_t s) {
    if (!pairdist_i8_has(f) || !aligned16(v) || (ld % 4) != 0 || d < 64 * kTK || d >= (int64_t(1) << 31)) return 1;
    const Scratch sc = carve(ws, f);
    // <rows, converter warps, copies, rows per box, boxes in the ring, tiles per step>
    if (f == 25) return launch_i8<25, 25, 1, 25, 6, 4>(v, d, ld, 0, nullptr, 0, dist, sc.tpart, sc.info, flag, force, s);
    return launch_i8<49, 25, 1, 49, 3, 2>(v, d, ld, 0, nullptr, 0, dist, sc.tpart, sc.info, flag, force, s);
}

// The same from the replicas: vote (Eq. 3) and distances in one pass; the winners go to `voted`.
int vote_pairdist_i8(const float* rep, int r, int f, int64_t d, int64_t ld_file, int64_t ld_rep, float* voted, int64_t ld_voted,
                     double* dist, void* ws, int* flag, int force, cudaStream_t s) {
    if (!pairdist_i8_has(f) || !aligned16(rep) || !aligned16(voted) || (ld_file % 4) != 0 || (ld_rep % 4) != 0 ||
        (ld_voted % 4) != 0 || d < 64 * kTK || d >= (int64_t(1) << 31))
        return 1;
    const Scratch sc = carve(ws, f);
#define BZ_I8_CASE(R_, F_, W_, FC_, NS_, TS_) \
    if (r == R_ && f == F_)                   \
        return launch_i8<F_, W_, R_, FC_, NS_, TS_>(rep, d, ld_file, ld_rep, voted, ld_voted, dist, sc.tpart, sc.info, flag, force, s);
    // with the copies in front the kernel is bound by HBM: where shared memory forces the choice, a third box in
    // flight is worth more than a second tile per step (r = 3, f = 49: 1.45 -> 1.32 ms; r = 7: 2.95 -> 2.65 ms)
    BZ_I8_CASE(3, 25, 25, 25, 3, 2)
    BZ_I8_CASE(3, 49, 25, 25, 3, 1)
    BZ_I8_CASE(5, 25, 25, 25, 2, 2)
    BZ_I8_CASE(5, 49, 25, 25, 2, 1)
    BZ_I8_CASE(7, 49, 13, 13, 3, 1)
#undef BZ_I8_CASE
    return 1;
}

int pairdist_i8_stall(int on) {
    const int v = on ? 1 : 0;
    const cudaError_t e = cudaMemcpyToSymbol(g_i8_stall, &v, sizeof(int));
    return e == cudaSuccess ? BZ_OK : cuda_failed(e);
}

int pairdist_i8_timeouts(unsigned int* count) {
    const cudaError_t e = cudaMemcpyFromSymbol(count, g_i8_timeouts, sizeof(unsigned int));
    return e == cudaSuccess ? BZ_OK : cuda_failed(e);
}

}  // namespace bz
