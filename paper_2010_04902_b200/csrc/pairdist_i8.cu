// Pairwise squared distances of the Krum family (Sec. 1.2; cost in Appendix A.1) on the tensor cores,
// in exact integer arithmetic.  Host side; the kernel is in pairdist_i8_kernel.cuh.
#include "pairdist_i8_kernel.cuh"

namespace bz {

namespace {

// After the main kernel, ONE small kernel of F CTAs finishes the job (three launches cost three times the latency of
// a dependent launch, which at a million coordinates was a fifth of the call):
//   every CTA: D^ for its share of the pairs from the CTAs' partial matrices; the exact contribution of the
//              outlier coordinates listed for "its" row; that row's rounding budget N_a^2; the CTAs' marks;
//   the CTA that finishes last (a ticket counter, no waiting): the bound on the conversion error -> final
//              distances, flag[0], flag[1].
// flag[0] = 1 asks for the binary64 kernel: the bound does not fit the tolerance (ignored with force != 0), a
// row holds values the fixed-point scale cannot carry, an outlier list overflowed, or a CTA stopped early.
// flag[1] = 1 says the latter: a bounded wait ran out, the partial matrices are incomplete and so are the voted
// rows of the kernel with the vote in front.
constexpr double kRelTol = 1e-7;   // the library's tolerance for a squared distance
constexpr int kFinishThreads = 1024;   // 32 warps: with F CTAs every pair has a warp of its own, and the last CTA covers the matrix in three sweeps

__device__ __forceinline__ double ld_l2(const double* p) { return __ldcg(p); }

// One warp per pair a <= b: lane l takes CTAs l, l+32, ... in order, then the lanes are added in a fixed
// tree.  Identical rows meet identical numbers in the same order and get identical distances.  The diagonal
// pairs deliver |q_a|^2 (what the binary64 sums had to carry: the bound covers their rounding with it).
template <int F>
__device__ __forceinline__ void finish_reduce_pair(const double* __restrict__ tpart, int n_ctas, int a, int b, int lane,
                                                   double* __restrict__ dist, double* __restrict__ norm2) {
    // at most kNumSMs partial matrices: five per lane, all loads in flight at once, added in the order c = lane, lane + 32, ...
    constexpr int kPerLane = (kNumSMs + 31) / 32;
    double t[kPerLane];
#pragma unroll
    for (int k = 0; k < kPerLane; ++k) {
        const int c = lane + 32 * k;
        t[k] = 0.0;
        if (c < n_ctas) {
            const double* T = tpart + static_cast<size_t>(c) * F * F;
            t[k] = a < b ? (T[a * F + a] + T[b * F + b]) - (T[a * F + b] + T[b * F + a]) : T[a * F + a];
        }
    }
    double s = 0.0;
#pragma unroll
    for (int k = 0; k < kPerLane; ++k)
        if (lane + 32 * k < n_ctas) s += t[k];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
    if (lane == 0) {
        if (a < b) {
            dist[a * F + b] = s;
            dist[b * F + a] = s;
        } else {
            dist[a * F + a] = 0.0;
            norm2[a] = s;
        }
    }
}

struct FinishShared {
    int cnt[kNumSMs], off[kNumSMs + 1];
    int j[kNumSMs * kOutCap];
    short c[kNumSMs * kOutCap];
};

// What the listed outlier coordinates contribute.  The CTA handles row a's lists, thread b the pair (a, b):
//   corr[a][b] = sum over row a's outliers j of (v_a[j] - v_b[j])^2 - (0 - fed_b[j])^2
// with fed_b[j] what row b fed the contraction at j: its value, or zero if j is on row b's list too (then the
// pair is handled from the list of the lower row only).  Lists are walked CTA by CTA, entry by entry:
// a fixed order.  The last CTA adds corr[a][b] + corr[b][a] to D^.  (Block-uniform control flow.)
template <int F>
__device__ __forceinline__ void finish_outliers(FinishShared& sh, const float* __restrict__ v, int64_t ld, const int* __restrict__ info,
                                                const int* __restrict__ olist, int n_ctas, int a, double* __restrict__ corr) {
    const int tid = threadIdx.x;
    int mine = 0;
    for (int c = tid; c < n_ctas; c += blockDim.x) {
        const int n = info[c * kInfoStride + kInfoOut + a];
        sh.cnt[c] = n > kOutCap ? kOutCap : (n < 0 ? 0 : n);  // an overflowing list sends the caller to the binary64 kernel anyway
        mine |= sh.cnt[c];
    }
    if (!__syncthreads_or(mine)) {  // nearly always: no CTA listed anything for this row
        if (tid < F) corr[a * F + tid] = 0.0;
        return;
    }
    // offsets of the CTAs' lists in the compact list: thread c adds the counts before its own
    for (int c = tid; c <= n_ctas; c += blockDim.x) {
        int run = 0;
        for (int k = 0; k < c; ++k) run += sh.cnt[k];
        sh.off[c] = run;
    }
    __syncthreads();
    const int total = sh.off[n_ctas];
    // row a's entries, CTA by CTA, in list order
    for (int e = tid; e < n_ctas * kOutCap; e += blockDim.x) {
        const int c = e / kOutCap, k = e % kOutCap;
        if (k < sh.cnt[c]) {
            sh.j[sh.off[c] + k] = olist[(static_cast<size_t>(c) * 64 + a) * kOutCap + k];
            sh.c[sh.off[c] + k] = static_cast<short>(c);
        }
    }
    __syncthreads();
    const int b = tid;
    if (b >= F) return;
    double sum = 0.0;
    if (b != a) {
#pragma unroll 4
        for (int e = 0; e < total; ++e) {
            const int64_t j = sh.j[e];
            const int c = sh.c[e];
            const float va = v[a * ld + j], vb = v[b * ld + j];
            // did row b enter as zero at j as well?  Then j is on its list in the same CTA.
            int n_b = info[c * kInfoStride + kInfoOut + b];
            n_b = n_b > kOutCap ? kOutCap : n_b;
            bool b_out = false;
            const int* list_b = olist + (static_cast<size_t>(c) * 64 + b) * kOutCap;
            for (int k = 0; k < n_b; ++k) b_out = b_out || list_b[k] == static_cast<int>(j);
            const double diff = static_cast<double>(va) - static_cast<double>(vb);
            const double fed = b_out ? 0.0 : static_cast<double>(vb);
            if (!(b_out && b < a)) sum += diff * diff - fed * fed;
        }
    }
    corr[a * F + b] = sum;
}

// The bound and the marks -> final distances, flag[0], flag[1] (the last CTA).
//   N_a^2 = sum over CTAs (and a row's successive scales) of n_small * (step / 2)^2, step = 2^(E - 30): every rounded
//   value moved by at most half a step
//   |D^ - D~| <= 2 (N_a + N_b) sqrt(D^) + (N_a + N_b)^2, D~ the distance with the outliers as zeros (Cauchy-Schwarz)
//   + 2^-39 (|q_a|^2 + |q_b|^2) for the binary64 sums behind D^ (a few thousand roundings of terms of that size)
// must stay below kRelTol times the final distance D^ + corr.
template <int F>
__global__ void __launch_bounds__(kFinishThreads)
    pairdist_i8_finish_kernel(const double* __restrict__ tpart, const float* __restrict__ v, int64_t ld, int* __restrict__ info,
                              const int* __restrict__ olist, int n_ctas, double* __restrict__ dist, double* __restrict__ corr,
                              double* __restrict__ norm2, double* __restrict__ n2_rows, int force, int* __restrict__ flag) {
    __shared__ FinishShared sh;
    constexpr int kParts = 16;
    __shared__ double s_part[kParts];
    __shared__ int s_last;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, row = blockIdx.x;
    // ---- this CTA's share of the pairs a <= b: pair numbers row, row + F, ... (rows of the upper triangle in order)
    constexpr int kPairs = F * (F + 1) / 2;
    for (int p = row + F * warp; p < kPairs; p += F * (kFinishThreads / 32)) {
        int a = 0, rem = p;
        while (rem >= F - a) {
            rem -= F - a;
            ++a;
        }
        finish_reduce_pair<F>(tpart, n_ctas, a, a + rem, lane, dist, norm2);
    }
    // ---- row `row`: rounding budget (sixteen threads, each over every sixteenth CTA in order; their sums are
    // added in a fixed order) and the CTAs' marks
    int marks = 0;
    if (tid < kParts) {
        double n2 = 0.0;
#pragma unroll 5
        for (int c = tid; c < n_ctas; c += kParts) {
            const int* rec = info + c * kInfoStride;
            const double half_step = __longlong_as_double(static_cast<long long>(1023 + rec[kInfoE + row] - 31) << 52);
            n2 += reinterpret_cast<const double*>(rec + kInfoN2)[row] + static_cast<double>(rec[kInfoSmall + row]) * half_step * half_step;
            if (rec[kInfoOut + row] > kOutCap) marks |= kBadValues;
        }
        s_part[tid] = n2;
    }
    if (row == 0)
        for (int c = tid; c < n_ctas; c += kFinishThreads) marks |= info[c * kInfoStride + kInfoBad];
    if (marks) atomicOr(&info[kInfoMarks], marks);
    // ---- row `row`: its outliers (syncs inside: also orders s_part)
    finish_outliers<F>(sh, v, ld, info, olist, n_ctas, row, corr);
    __syncthreads();
    if (tid == 0) {
        double n2 = 0.0;
#pragma unroll
        for (int part = 0; part < kParts; ++part) n2 += s_part[part];
        n2_rows[row] = n2;
    }
    // ---- the last CTA to get here sees what all the others wrote (fence, ticket, fence)
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = atomicAdd(&info[kInfoTicket], 1) == F - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    __shared__ double s_n[F], s_norm2[F], s_min_nz[F], s_zero_n2[F];
    __shared__ int s_bad;
    if (tid == 0) s_bad = 0;
    if (tid < F) {
        s_n[tid] = sqrt(ld_l2(n2_rows + tid));
        s_norm2[tid] = ld_l2(norm2 + tid);
        s_min_nz[tid] = 1e300;
        s_zero_n2[tid] = 0.0;
    }
    __syncthreads();
    bool bad = false;
    constexpr int kSweeps = (F * F + kFinishThreads - 1) / kFinishThreads;
    double dh_[kSweeps], c1_[kSweeps], c2_[kSweeps];
#pragma unroll
    for (int k = 0; k < kSweeps; ++k) {  // all loads first: one trip to L2, not three
        const int p = tid + k * kFinishThreads;
        const int a = p / F, b = p % F;
        dh_[k] = c1_[k] = c2_[k] = 0.0;
        if (p < F * F && a < b) {
            dh_[k] = ld_l2(dist + a * F + b);
            c1_[k] = ld_l2(corr + a * F + b);
            c2_[k] = ld_l2(corr + b * F + a);
        }
    }
#pragma unroll
    for (int k = 0; k < kSweeps; ++k) {
        const int p = tid + k * kFinishThreads;
        const int a = p / F, b = p % F;
        if (p >= F * F || a >= b) continue;
        const double dh = dh_[k];
        const double df = dh + (c1_[k] + c2_[k]);
        const double n = s_n[a] + s_n[b];
        if (!(dh >= 0.0) || !(df >= 0.0)) {
            bad = true;
        } else {
            const double err = 2.0 * n * sqrt(dh) + n * n + 1.8189894035458565e-12 * (s_norm2[a] + s_norm2[b]);
            if (df > 0.0) {
                if (err > kRelTol * df) bad = true;
                atomicMin(reinterpret_cast<unsigned long long*>(&s_min_nz[a]), static_cast<unsigned long long>(__double_as_longlong(df)));
                atomicMin(reinterpret_cast<unsigned long long*>(&s_min_nz[b]), static_cast<unsigned long long>(__double_as_longlong(df)));
            } else {
                // rows that convert to the same integers may still differ, by up to err: judged below against the
                // smallest distance either row has to anything else
                atomicMax(reinterpret_cast<unsigned long long*>(&s_zero_n2[a]), static_cast<unsigned long long>(__double_as_longlong(err)));
                atomicMax(reinterpret_cast<unsigned long long*>(&s_zero_n2[b]), static_cast<unsigned long long>(__double_as_longlong(err)));
            }
        }
        dist[a * F + b] = df;
        dist[b * F + a] = df;
    }
    if (bad) atomicOr(&s_bad, 1);
    __syncthreads();
    if (tid < F && s_zero_n2[tid] > 0.0 && s_min_nz[tid] < 1e300 && s_zero_n2[tid] > kRelTol * s_min_nz[tid]) atomicOr(&s_bad, 1);
    __syncthreads();
    if (tid == 0) {
        const int all_marks = atomicOr(&info[kInfoMarks], 0);
        flag[0] = ((s_bad && !force) || all_marks) ? 1 : 0;
        flag[1] = (all_marks & kBadStopped) ? 1 : 0;
    }
}

struct Scratch {
    double* tpart;
    int* info;
    int* olist;
    double* corr;
    double* norm2;
    double* n2;
};

// rep: R = 1: rows [f][d] with leading dimension ld_file.  R > 1: replicas[r][f][d].
// Returns 1 if the tensor map cannot express the shape.
template <int F, int W, int R, int FC, int NS, int TS>
int launch_i8(const float* rep, int64_t d, int64_t ld_file, int64_t ld_rep, float* voted, int64_t ld_voted, double* dist,
              const Scratch& sc, int* flag, int force, cudaStream_t s) {
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
    kern<<<static_cast<int>(ctas), S::kThreads, S::kSmem, s>>>(map, d, voted, ld_voted, sc.tpart, sc.info, sc.olist);
    note_launch();
    int st = check_launch();
    if (st != BZ_OK) return st;
    // the rows the contraction saw: the given ones, or the winners the kernel has just written
    const float* rows = R > 1 ? voted : rep;
    const int64_t ld_rows = R > 1 ? ld_voted : ld_file;
    pairdist_i8_finish_kernel<F><<<F, kFinishThreads, 0, s>>>(sc.tpart, rows, ld_rows, sc.info, sc.olist, static_cast<int>(ctas), dist,
                                                            sc.corr, sc.norm2, sc.n2, force, flag);
    note_launch();
    return check_launch();
}

size_t tpart_bytes(int f) { return round_up(static_cast<size_t>(kNumSMs) * f * f * sizeof(double), 256); }
size_t info_bytes() { return round_up(static_cast<size_t>(kNumSMs) * kInfoStride * sizeof(int), 256); }
size_t olist_bytes() { return round_up(static_cast<size_t>(kNumSMs) * 64 * kOutCap * sizeof(int), 256); }
size_t corr_bytes(int f) { return round_up(static_cast<size_t>(f) * f * sizeof(double), 256); }
size_t norm_bytes() { return round_up(2 * 64 * sizeof(double), 256); }   // |q_a|^2 and N_a^2 per row

Scratch carve(void* ws, int f) {
    char* p = static_cast<char*>(ws);
    Scratch s;
    s.tpart = reinterpret_cast<double*>(p);
    p += tpart_bytes(f);
    s.info = reinterpret_cast<int*>(p);
    p += info_bytes();
    s.olist = reinterpret_cast<int*>(p);
    p += olist_bytes();
    s.corr = reinterpret_cast<double*>(p);
    p += corr_bytes(f);
    s.norm2 = reinterpret_cast<double*>(p);
    s.n2 = s.norm2 + 64;
    return s;
}

}  // namespace

bool pairdist_i8_has(int f) { return f == 25 || f == 49; }

// bytes of the partial matrices, the per-CTA records, the outlier lists and their corrections
size_t pairdist_i8_workspace(int f) {
    if (!pairdist_i8_has(f)) return 0;
    return tpart_bytes(f) + info_bytes() + olist_bytes() + corr_bytes(f) + norm_bytes();
}

// Returns BZ_OK / an error, or 1 when this path does not apply (shape, alignment, size).  On BZ_OK
// dist holds the distances, flag[0] (device) is 1 if they must be recomputed in binary32 and flag[1] is 1
// if the kernel stopped early.
int pairdist_i8(const float* v, int f, int64_t d, int64_t ld, double* dist, void* ws, int* flag, int force, cudaStream_t s) {
    if (!pairdist_i8_has(f) || !aligned16(v) || (ld % 4) != 0 || d < 64 * kTK || d >= (int64_t(1) << 31)) return 1;
    const Scratch sc = carve(ws, f);
    // <rows, converter warps, copies, rows per box, boxes in the ring, tiles per step>
    if (f == 25) return launch_i8<25, 25, 1, 25, 6, 4>(v, d, ld, 0, nullptr, 0, dist, sc, flag, force, s);
    return launch_i8<49, 25, 1, 49, 3, 2>(v, d, ld, 0, nullptr, 0, dist, sc, flag, force, s);
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
        return launch_i8<F_, W_, R_, FC_, NS_, TS_>(rep, d, ld_file, ld_rep, voted, ld_voted, dist, sc, flag, force, s);
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
