// The Krum family on the f voted gradients (Sec. 1.2, Sec. 6.1): Multi-Krum selection and mean,
// Bulyan's iterated selection and its trimmed mean around the median, and the end-to-end calls.
// The pairwise distances they start from are in pairdist.cu.
#include "bz_common.cuh"

namespace bz {

// pairdist.cu
size_t pairdist_workspace(int f);
size_t krum_workspace_bytes(int op, int f);
int pairdist_on_device(const float* v, int f, int64_t d, int64_t ld, double* dist, void* ws, cudaStream_t s, bool tensor_cores);
int validate_rows(const float* v, int f, int64_t d, int64_t ld);
int check_workspace(void* ws, size_t have, size_t need);

namespace {

// ------------------------------------------------------------------------------------------------
// Selection kernels: one CTA, thread a owns row a.

// Row a's distances to the other rows, ascending (insertion sort in local memory; f <= BZ_MAX_F).
// The loads are issued first, all independent; the order of a row never changes afterwards.
struct SortedRow {
    double val[BZ_MAX_F];
    unsigned char idx[BZ_MAX_F];
    int n;
};
__device__ void sort_row(const double* __restrict__ dist, int f, int a, SortedRow& row) {
    for (int b = 0; b < f; ++b) row.val[b] = dist[a * f + b];
    int n = 0;
    // in place: entries 0 .. n-1 are sorted, entry b is still raw (b >= n always holds)
    for (int b = 0; b < f; ++b) {
        if (b == a) continue;
        const double x = row.val[b];
        int pos = n++;
        while (pos > 0 && row.val[pos - 1] > x) {
            row.val[pos] = row.val[pos - 1];
            row.idx[pos] = row.idx[pos - 1];
            --pos;
        }
        row.val[pos] = x;
        row.idx[pos] = static_cast<unsigned char>(b);
    }
    row.n = n;
}
// Krum score inside the rows flagged in `active`: the nb smallest distances to the other active rows,
// added in ascending order.
__device__ double krum_score(const SortedRow& row, const unsigned char* active, int nb) {
    double s = 0.0;
    int taken = 0;
    for (int t = 0; t < row.n && taken < nb; ++t)
        if (active[row.idx[t]]) {
            s += row.val[t];
            ++taken;
        }
    return s;
}

__global__ void __launch_bounds__(BZ_MAX_F) krum_select_kernel(const double* __restrict__ dist, int f, int c, int m,
                                                               int32_t* __restrict__ selected) {
    __shared__ double score[BZ_MAX_F];
    __shared__ unsigned char active[BZ_MAX_F];
    const int a = threadIdx.x;
    if (a < f) active[a] = 1;
    __syncthreads();
    if (a < f) {
        SortedRow row;
        sort_row(dist, f, a, row);
        score[a] = krum_score(row, active, f - c - 2);
    }
    __syncthreads();
    if (a < f) {
        int rank = 0;
        for (int b = 0; b < f; ++b) rank += (score[b] < score[a]) || (score[b] == score[a] && b < a);
        if (rank < m) selected[rank] = a;
    }
}

__global__ void __launch_bounds__(BZ_MAX_F) bulyan_select_kernel(const double* __restrict__ dist, int f, int c,
                                                                 int32_t* __restrict__ selected) {
    __shared__ double score[BZ_MAX_F];
    __shared__ unsigned char active[BZ_MAX_F];
    const int a = threadIdx.x;
    if (a < f) active[a] = 1;
    SortedRow row;
    row.n = 0;
    if (a < f) sort_row(dist, f, a, row);
    __syncthreads();
    const int theta = f - 2 * c;
    for (int t = 0; t < theta; ++t) {
        const int n = f - t;
        int nb = n - c - 2;
        if (nb < 1) nb = 1;
        if (nb > n - 1) nb = n - 1;
        if (a < f && active[a]) score[a] = (n > 1) ? krum_score(row, active, nb) : 0.0;
        __syncthreads();
        bool win = false;
        if (a < f && active[a]) {
            win = true;
            for (int b = 0; b < f; ++b)
                if (b != a && active[b] && ((score[b] < score[a]) || (score[b] == score[a] && b < a))) win = false;
        }
        __syncthreads();
        if (win) {
            selected[t] = a;
            active[a] = 0;
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------------
// The same selections for f <= 64 with the sorted rows in shared memory.
// Sorting is by rank counting: the matrix is staged in shared memory and every thread counts, for a few entries
// (a, b), how many of row a's distances precede its own (by value, then index).  A score is the sum of the first
// nb ACTIVE entries of the sorted row, added one by one in ascending order - the same sums in the same order as
// in the kernels above; one warp per row forms it.
constexpr int kSelF = 64;
constexpr int kSelWarps = 32;

struct SelectShared {
    double raw[kSelF][kSelF];
    double sval[kSelF][kSelF];
    double comp[kSelWarps][kSelF];
    double score[kSelF];
    unsigned char sidx[kSelF][kSelF];
    unsigned char active[kSelF];
};

__device__ __forceinline__ void sort_rows_shared(const double* __restrict__ dist, int f, SelectShared& sh) {
    for (int e = threadIdx.x; e < f * f; e += blockDim.x) sh.raw[e / f][e % f] = dist[e];
    __syncthreads();
    for (int e = threadIdx.x; e < f * f; e += blockDim.x) {
        const int a = e / f, b = e % f;
        if (b == a) continue;
        const double x = sh.raw[a][b];
        int rank = 0;
#pragma unroll 8
        for (int b2 = 0; b2 < f; ++b2) {
            const double y = sh.raw[a][b2];
            rank += (b2 != a) && ((y < x) || (y == x && b2 < b));
        }
        sh.sval[a][rank] = x;
        sh.sidx[a][rank] = static_cast<unsigned char>(b);
    }
}

// warp-collective: score of row a among the active rows (the result is valid in lane 0).
// The lanes compact the first nb active entries into `comp` (positions by prefix counts of the
// ballots); lane 0 adds them in ascending order.
__device__ __forceinline__ double krum_score_warp(const SelectShared& sh, int f, int a, int nb, double* comp) {
    const int lane = threadIdx.x & 31;
    const int p0 = lane, p1 = lane + 32;
    const bool act0 = p0 < f - 1 && sh.active[sh.sidx[a][p0]];
    const bool act1 = p1 < f - 1 && sh.active[sh.sidx[a][p1]];
    const unsigned m0 = __ballot_sync(0xffffffffu, act0), m1 = __ballot_sync(0xffffffffu, act1);
    const unsigned below = (1u << lane) - 1u;
    const int q0 = __popc(m0 & below), q1 = __popc(m0) + __popc(m1 & below);
    if (act0 && q0 < nb) comp[q0] = sh.sval[a][p0];
    if (act1 && q1 < nb) comp[q1] = sh.sval[a][p1];
    __syncwarp();
    double s = 0.0;
    if (lane == 0) {
        const int total = min(nb, __popc(m0) + __popc(m1));
#pragma unroll 4
        for (int k = 0; k < total; ++k) s += comp[k];
    }
    __syncwarp();
    return s;
}

// bulyan == 0: Multi-Krum (first m of the ranking); bulyan != 0: theta = f - 2c picks, one per round
__global__ void __launch_bounds__(kSelWarps * 32) select_shared_kernel(const double* __restrict__ dist, int f, int c, int m, int bulyan,
                                                             int32_t* __restrict__ selected) {
    extern __shared__ __align__(16) unsigned char select_smem[];
    SelectShared& sh = *reinterpret_cast<SelectShared*>(select_smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid < f) sh.active[tid] = 1;
    sort_rows_shared(dist, f, sh);
    __syncthreads();
    if (!bulyan) {
        for (int a = warp; a < f; a += kSelWarps) {
            const double s = krum_score_warp(sh, f, a, f - c - 2, sh.comp[warp]);
            if (lane == 0) sh.score[a] = s;
        }
        __syncthreads();
        if (tid < f) {
            int rank = 0;
            for (int b = 0; b < f; ++b) rank += (sh.score[b] < sh.score[tid]) || (sh.score[b] == sh.score[tid] && b < tid);
            if (rank < m) selected[rank] = tid;
        }
        return;
    }
    const int theta = f - 2 * c;
    for (int t = 0; t < theta; ++t) {
        const int n = f - t;
        int nb = n - c - 2;
        if (nb < 1) nb = 1;
        if (nb > n - 1) nb = n - 1;
        for (int a = warp; a < f; a += kSelWarps) {
            if (!sh.active[a]) continue;  // uniform over the warp
            const double s = (n > 1) ? krum_score_warp(sh, f, a, nb, sh.comp[warp]) : 0.0;
            if (lane == 0) sh.score[a] = s;
        }
        __syncthreads();
        if (warp == 0) {
            // smallest (score, index) among the active rows
            double best = 0.0;
            int who = -1;
            for (int a = lane; a < f; a += 32)
                if (sh.active[a] && (who < 0 || sh.score[a] < best)) {  // a grows: a tie keeps the lower index
                    best = sh.score[a];
                    who = a;
                }
            for (int o = 16; o > 0; o >>= 1) {
                const double ob = __shfl_down_sync(0xffffffffu, best, o);
                const int ow = __shfl_down_sync(0xffffffffu, who, o);
                if (ow >= 0 && (who < 0 || ob < best || (ob == best && ow < who))) {
                    best = ob;
                    who = ow;
                }
            }
            if (lane == 0) {
                selected[t] = who;
                sh.active[who] = 0;
            }
        }
        __syncthreads();
    }
}

int launch_select_shared(const double* dist, int f, int c, int m, int bulyan, int32_t* selected, cudaStream_t s) {
    // per device, so set on every call (it is a host-side table entry, not a launch)
    const cudaError_t attr = cudaFuncSetAttribute(select_shared_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                  static_cast<int>(sizeof(SelectShared)));
    if (attr != cudaSuccess) return cuda_failed(attr);
    select_shared_kernel<<<1, kSelWarps * 32, sizeof(SelectShared), s>>>(dist, f, c, m, bulyan, selected);
    return BZ_OK;
}

// ------------------------------------------------------------------------------------------------
// Means over selected rows.

template <typename V> struct FL;
template <> struct FL<float4> { static constexpr int n = 4; };
template <> struct FL<float> { static constexpr int n = 1; };

template <typename V>
__global__ void __launch_bounds__(256) mean_rows_kernel(const V* __restrict__ v, int64_t n, int64_t ld,
                                                        const int32_t* __restrict__ selected, int m, V* __restrict__ out) {
    __shared__ int32_t sel[BZ_MAX_F];
    for (int t = threadIdx.x; t < m; t += blockDim.x) sel[t] = selected[t];
    __syncthreads();
    const double dm = static_cast<double>(m);
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; j < n; j += stride) {
        if constexpr (FL<V>::n == 4) {
            double s0 = 0, s1 = 0, s2 = 0, s3 = 0;
#pragma unroll 4
            for (int t = 0; t < m; ++t) {
                const float4 x = __ldcs(v + sel[t] * ld + j);
                s0 += x.x; s1 += x.y; s2 += x.z; s3 += x.w;
            }
            out[j] = make_float4(static_cast<float>(s0 / dm), static_cast<float>(s1 / dm),
                                 static_cast<float>(s2 / dm), static_cast<float>(s3 / dm));
        } else {
            double s = 0;
            for (int t = 0; t < m; ++t) s += v[sel[t] * ld + j];
            out[j] = static_cast<float>(s / dm);
        }
    }
}

// The window grown one value at a time, as the definition states it: the neighbour (below or above) that is
// closer to the median in binary32 enters, the lower one on ties.  Used as written by the run-time-theta kernel
// and, out of line, by the register kernels for columns that hold an infinity or a NaN (a comparison with a NaN
// distance is false, which takes the upper neighbour).
__device__ __noinline__ float window_mean_stepwise(const float* s, int theta, int beta) {
    const int mid = (theta - 1) / 2;
    const float med = s[mid];
    int lo = mid, hi = mid;
    while (hi - lo + 1 < beta) {
        const bool can_lo = lo > 0, can_hi = hi < theta - 1;
        bool take_lo = can_lo;
        if (can_lo && can_hi) take_lo = fabsf(__fsub_rn(s[lo - 1], med)) <= fabsf(__fsub_rn(s[hi + 1], med));
        if (take_lo) --lo; else ++hi;
    }
    double sum = 0.0;
    for (int t = lo; t <= hi; ++t) sum += static_cast<double>(s[t]);
    return static_cast<float>(sum / static_cast<double>(beta));
}

// sum += x if (du >= dl) == GE, as one compare and one predicated addition (finite values: "not >=" is "<").
// The test is made where it is used, twice per pair, so that no flag has to live across the other additions:
// a thread has seven predicate registers, and a flag parked in a general register costs more than the second compare.
template <bool GE> __device__ __forceinline__ void add_if(double& sum, float x, float du, float dl) {
    if constexpr (GE)
        asm("{\n\t.reg .pred p;\n\t.reg .f64 xd;\n\tsetp.ge.f32 p, %2, %3;\n\tcvt.f64.f32 xd, %1;\n\t@p add.rn.f64 %0, %0, xd;\n\t}"
            : "+d"(sum) : "f"(x), "f"(du), "f"(dl));
    else
        asm("{\n\t.reg .pred p;\n\t.reg .f64 xd;\n\tsetp.lt.f32 p, %2, %3;\n\tcvt.f64.f32 xd, %1;\n\t@p add.rn.f64 %0, %0, xd;\n\t}"
            : "+d"(sum) : "f"(x), "f"(du), "f"(dl));
}

// Window of the BETA sorted values closest to the median, without the steps.  With finite values the two
// sequences of distances ascend, so growing the window merges them: the p-th lower value enters before the
// q-th upper one iff its distance is not larger, hence it belongs to the window iff the (BETA-p)-th upper value
// does not exist or is at least as far.  Of each such pair exactly one is in the window (it holds BETA-1 values
// besides the median), so the tests themselves decide membership and no window bounds are formed.
// s[] ascending, sorted with the binary32 comparators, which leave every infinity at an end and a NaN at both:
// for those columns the function returns false (the caller takes the steps, from the column itself).
// mean: the mean of the window (binary64 sum, ascending).
template <int THETA, int BETA> __device__ __forceinline__ bool window_mean(const float (&s)[THETA], float& mean) {
    constexpr int MID = (THETA - 1) / 2;
    constexpr float kInf = __builtin_huge_valf();
    if (!(fabsf(s[0]) < kInf && fabsf(s[THETA - 1]) < kInf)) return false;
    const float med = s[MID];
    // ascending positions: the lower values (p = distance in rank from the median, descending), the median, the
    // upper values (u ascending, paired with the lower value p = BETA - u)
    double sum = 0.0;
#pragma unroll
    for (int p = (MID < BETA - 1 ? MID : BETA - 1); p >= 1; --p) {
        const int up = MID + (BETA - p);  // index of the (BETA-p)-th upper value
        if (up > THETA - 1)
            sum += static_cast<double>(s[MID - p]);
        else
            add_if<true>(sum, s[MID - p], fabsf(__fsub_rn(s[up], med)), fabsf(__fsub_rn(s[MID - p], med)));
    }
    sum += static_cast<double>(med);
#pragma unroll
    for (int u = 1; u <= BETA - 1 && MID + u <= THETA - 1; ++u) {
        const int p = BETA - u;
        if (p > MID)  // no lower value competes with it
            sum += static_cast<double>(s[MID + u]);
        else
            add_if<false>(sum, s[MID + u], fabsf(__fsub_rn(s[MID + u], med)), fabsf(__fsub_rn(s[MID - p], med)));
    }
    mean = static_cast<float>(sum / static_cast<double>(BETA));
    return true;
}

// One coordinate, out of line: the column is read again, sorted in the total order (insertion sort on order keys in
// local memory) and its window grown step by step.  For the columns the register kernels hand back: those that
// hold an infinity or a NaN.
__device__ __noinline__ float trimmed_column_stepwise(const float* __restrict__ v, const int64_t* row, int64_t j, int theta, int beta) {
    int k[BZ_MAX_F];
    for (int t = 0; t < theta; ++t) {
        const int x = order_key(__float_as_uint(v[row[t] + j]));
        int pos = t;
        while (pos > 0 && k[pos - 1] > x) {
            k[pos] = k[pos - 1];
            --pos;
        }
        k[pos] = x;
    }
    float sorted[BZ_MAX_F];
    for (int t = 0; t < theta; ++t) sorted[t] = __uint_as_float(key_bits(k[t]));
    return window_mean_stepwise(sorted, theta, beta);
}

// V coordinates per thread (V = 2, 4: 64- and 128-bit loads, rows aligned accordingly): the address arithmetic
// and the load instructions are shared by the V coordinates.
template <int THETA, int BETA, int V>
__global__ void __launch_bounds__(128) trimmed_mean_kernel(const float* __restrict__ v, int64_t d, int64_t ld,
                                                           const int32_t* __restrict__ selected,
                                                           float* __restrict__ out) {
    __shared__ int64_t row[THETA];
    for (int t = threadIdx.x; t < THETA; t += blockDim.x) row[t] = selected[t] * ld;
    __syncthreads();
    const int64_t groups = (d + V - 1) / V;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t g = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; g < groups; g += stride) {
        const int64_t j = g * V;
        float k[V][THETA];
        const bool whole = j + V <= d;  // the last group may hold fewer coordinates
        if (V == 4 && whole) {
#pragma unroll
            for (int t = 0; t < THETA; ++t) {
                const float4 x = __ldcs(reinterpret_cast<const float4*>(v + row[t] + j));
                k[0][t] = x.x;
                k[V > 1 ? 1 : 0][t] = x.y;
                k[V > 2 ? 2 : 0][t] = x.z;
                k[V > 3 ? 3 : 0][t] = x.w;
            }
        } else if (V == 2 && whole) {
#pragma unroll
            for (int t = 0; t < THETA; ++t) {
                const float2 x = __ldcs(reinterpret_cast<const float2*>(v + row[t] + j));
                k[0][t] = x.x;
                k[V > 1 ? 1 : 0][t] = x.y;
            }
        } else {
#pragma unroll
            for (int c = 0; c < V; ++c) {
                const int64_t jc = j + c < d ? j + c : d - 1;  // past the end: the last coordinate once more
#pragma unroll
                for (int t = 0; t < THETA; ++t) k[c][t] = __ldcs(v + row[t] + jc);
            }
        }
        float res[V];
#pragma unroll
        for (int c = 0; c < V; ++c) {
            // Finite columns (all but a handful) sort as numbers: no order keys, half the operations of a comparator on
            // keys with its max on the other pipe.  The kernel is bound by the ALU pipe and by instruction issue.
            SortNet<THETA>::run(k[c]);
            if (!window_mean<THETA, BETA>(k[c], res[c])) {
                const int64_t jc = j + c < d ? j + c : d - 1;
                res[c] = trimmed_column_stepwise(v, row, jc, THETA, BETA);
            }
        }
        if (V == 4 && whole) {
            *reinterpret_cast<float4*>(out + j) = make_float4(res[0], res[V > 1 ? 1 : 0], res[V > 2 ? 2 : 0], res[V > 3 ? 3 : 0]);
        } else if (V == 2 && whole) {
            *reinterpret_cast<float2*>(out + j) = make_float2(res[0], res[V > 1 ? 1 : 0]);
        } else {
#pragma unroll
            for (int c = 0; c < V; ++c)
                if (j + c < d) out[j + c] = res[c];
        }
    }
}


// run-time theta: insertion sort in local memory, explicit window growth
__global__ void __launch_bounds__(128) trimmed_mean_generic_kernel(const float* __restrict__ v, int64_t d, int64_t ld,
                                                                   const int32_t* __restrict__ selected, int theta,
                                                                   int beta, float* __restrict__ out) {
    __shared__ int32_t sel[BZ_MAX_F];
    for (int t = threadIdx.x; t < theta; t += blockDim.x) sel[t] = selected[t];
    __syncthreads();
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; j < d; j += stride) {
        int k[BZ_MAX_F];
        for (int t = 0; t < theta; ++t) {
            const int x = order_key(__float_as_uint(v[sel[t] * ld + j]));
            int pos = t;
            while (pos > 0 && k[pos - 1] > x) {
                k[pos] = k[pos - 1];
                --pos;
            }
            k[pos] = x;
        }
        float sorted[BZ_MAX_F];
        for (int t = 0; t < theta; ++t) sorted[t] = __uint_as_float(key_bits(k[t]));
        out[j] = window_mean_stepwise(sorted, theta, beta);
    }
}

// ------------------------------------------------------------------------------------------------
// host side

int mean_rows_on_device(const float* v, int64_t d, int64_t ld, const int32_t* selected, int m, float* out,
                        cudaStream_t s) {
    const bool vec = aligned16(v) && aligned16(out) && (ld % 4 == 0);
    const int64_t n4 = vec ? d / 4 : 0;
    if (n4 > 0) {
        int64_t grid = (n4 + 255) / 256;
        if (grid > kNumSMs * 8) grid = kNumSMs * 8;
        mean_rows_kernel<float4><<<static_cast<int>(grid), 256, 0, s>>>(reinterpret_cast<const float4*>(v), n4, ld / 4,
                                                                        selected, m, reinterpret_cast<float4*>(out));
        note_launch();
        int st = check_launch();
        if (st != BZ_OK) return st;
    }
    const int64_t rest = d - 4 * n4;
    if (rest > 0) {
        int64_t grid = (rest + 255) / 256;
        if (grid > kNumSMs * 8) grid = kNumSMs * 8;
        mean_rows_kernel<float><<<static_cast<int>(grid), 256, 0, s>>>(v + 4 * n4, rest, ld, selected, m, out + 4 * n4);
        note_launch();
        return check_launch();
    }
    return BZ_OK;
}

template <int THETA, int BETA>
int launch_trimmed(const float* v, int64_t d, int64_t ld, const int32_t* selected, float* out, cudaStream_t s) {
    // widest loads the layout allows; four coordinates per thread only while their keys fit the registers
    const uintptr_t bits = reinterpret_cast<uintptr_t>(v) | reinterpret_cast<uintptr_t>(out) | static_cast<uintptr_t>(ld * 4);
    const int width = (THETA <= 25 && bits % 16 == 0) ? 4 : (bits % 8 == 0 ? 2 : 1);
    int64_t grid = ((d + width - 1) / width + 127) / 128;
    if (grid > kNumSMs * 16) grid = kNumSMs * 16;
    if (width == 4)
        trimmed_mean_kernel<THETA, BETA, (THETA <= 25 ? 4 : 2)><<<static_cast<int>(grid), 128, 0, s>>>(v, d, ld, selected, out);
    else if (width == 2)
        trimmed_mean_kernel<THETA, BETA, 2><<<static_cast<int>(grid), 128, 0, s>>>(v, d, ld, selected, out);
    else
        trimmed_mean_kernel<THETA, BETA, 1><<<static_cast<int>(grid), 128, 0, s>>>(v, d, ld, selected, out);
    note_launch();
    return check_launch();
}

// Register kernels exist for the (theta, beta) = (f - 2c, f - 4c) pairs of f = 25 and f = 49 (every c
// Bulyan admits) and a few small shapes; anything else runs the local-memory kernel.
int trimmed_mean_on_device(const float* v, int64_t d, int64_t ld, const int32_t* selected, int theta, int beta,
                           float* out, cudaStream_t s) {
#define BZ_TM_CASE(TH, BE) \
    if (theta == TH && beta == BE) return launch_trimmed<TH, BE>(v, d, ld, selected, out, s);
    BZ_TM_CASE(25, 25) BZ_TM_CASE(23, 21) BZ_TM_CASE(21, 17) BZ_TM_CASE(19, 13) BZ_TM_CASE(17, 9) BZ_TM_CASE(15, 5)
    BZ_TM_CASE(49, 49) BZ_TM_CASE(47, 45) BZ_TM_CASE(45, 41) BZ_TM_CASE(43, 37) BZ_TM_CASE(41, 33) BZ_TM_CASE(39, 29)
    BZ_TM_CASE(37, 25) BZ_TM_CASE(35, 21) BZ_TM_CASE(33, 17) BZ_TM_CASE(31, 13) BZ_TM_CASE(29, 9) BZ_TM_CASE(27, 5)
    BZ_TM_CASE(9, 9) BZ_TM_CASE(7, 5) BZ_TM_CASE(5, 3) BZ_TM_CASE(9, 1)
#undef BZ_TM_CASE
    int64_t grid = (d + 127) / 128;
    if (grid > kNumSMs * 8) grid = kNumSMs * 8;
    trimmed_mean_generic_kernel<<<static_cast<int>(grid), 128, 0, s>>>(v, d, ld, selected, theta, beta, out);
    note_launch();
    return check_launch();
}

}  // namespace

}  // namespace bz

using namespace bz;

extern "C" int bz_krum_select(const double* dist, int f, int c, int m, int32_t* selected, void* stream) {
    if (dist == nullptr || selected == nullptr || f < 1) return BZ_ERR_INVALID_ARG;
    if (f > BZ_MAX_F) return BZ_ERR_UNSUPPORTED;
    if (c < 0 || f < 2 * c + 3 || m < 1 || m > f) return BZ_ERR_PRECONDITION;
    if (f <= kSelF) {
        const int st = launch_select_shared(dist, f, c, m, 0, selected, static_cast<cudaStream_t>(stream));
        if (st != BZ_OK) return st;
    } else
        krum_select_kernel<<<1, BZ_MAX_F, 0, static_cast<cudaStream_t>(stream)>>>(dist, f, c, m, selected);
    note_launch();
    return check_launch();
}

extern "C" int bz_mean_rows(const float* voted, int f, int64_t d, int64_t ld, const int32_t* selected, int m,
                            float* out, void* stream) {
    int st = validate_rows(voted, f, d, ld);
    if (st != BZ_OK) return st;
    if (selected == nullptr || (out == nullptr && d > 0)) return BZ_ERR_INVALID_ARG;
    if (m < 1 || m > f) return BZ_ERR_PRECONDITION;
    if (d == 0) return BZ_OK;
    return mean_rows_on_device(voted, d, ld, selected, m, out, static_cast<cudaStream_t>(stream));
}

extern "C" int bz_multikrum(const float* voted, int f, int64_t d, int64_t ld, int c, int m, float* out,
                            int32_t* selected, double* dist, void* workspace, size_t workspace_bytes, void* stream) {
    int st = validate_rows(voted, f, d, ld);
    if (st != BZ_OK) return st;
    if ((out == nullptr && d > 0) || selected == nullptr) return BZ_ERR_INVALID_ARG;
    if (c < 0 || f < 2 * c + 3 || m < 1 || m > f) return BZ_ERR_PRECONDITION;
    st = check_workspace(workspace, workspace_bytes, krum_workspace_bytes(BZ_OP_MULTIKRUM, f));
    if (st != BZ_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    double* D = dist ? dist : reinterpret_cast<double*>(static_cast<char*>(workspace) + pairdist_workspace(f));
    st = pairdist_on_device(voted, f, d, ld, D, workspace, s, true);
    if (st != BZ_OK) return st;
    st = bz_krum_select(D, f, c, m, selected, stream);
    if (st != BZ_OK) return st;
    if (d == 0) return BZ_OK;
    return mean_rows_on_device(voted, d, ld, selected, m, out, s);
}

extern "C" int bz_bulyan_select(const double* dist, int f, int c, int32_t* selected, void* stream) {
    if (dist == nullptr || selected == nullptr || f < 1) return BZ_ERR_INVALID_ARG;
    if (f > BZ_MAX_F) return BZ_ERR_UNSUPPORTED;
    if (c < 0 || f < 4 * c + 3) return BZ_ERR_PRECONDITION;
    if (f <= kSelF) {
        const int st = launch_select_shared(dist, f, c, 0, 1, selected, static_cast<cudaStream_t>(stream));
        if (st != BZ_OK) return st;
    } else
        bulyan_select_kernel<<<1, BZ_MAX_F, 0, static_cast<cudaStream_t>(stream)>>>(dist, f, c, selected);
    note_launch();
    return check_launch();
}

extern "C" int bz_trimmed_mean(const float* voted, int f, int64_t d, int64_t ld, const int32_t* selected, int theta,
                               int beta, float* out, void* stream) {
    int st = validate_rows(voted, f, d, ld);
    if (st != BZ_OK) return st;
    if (selected == nullptr || (out == nullptr && d > 0)) return BZ_ERR_INVALID_ARG;
    if (theta < 1 || theta > f || beta < 1 || beta > theta) return BZ_ERR_PRECONDITION;
    if (d == 0) return BZ_OK;
    return trimmed_mean_on_device(voted, d, ld, selected, theta, beta, out, static_cast<cudaStream_t>(stream));
}

extern "C" int bz_bulyan(const float* voted, int f, int64_t d, int64_t ld, int c, float* out, int32_t* selected,
                         void* workspace, size_t workspace_bytes, void* stream) {
    int st = validate_rows(voted, f, d, ld);
    if (st != BZ_OK) return st;
    if ((out == nullptr && d > 0) || selected == nullptr) return BZ_ERR_INVALID_ARG;
    if (c < 0 || f < 4 * c + 3) return BZ_ERR_PRECONDITION;
    st = check_workspace(workspace, workspace_bytes, krum_workspace_bytes(BZ_OP_BULYAN, f));
    if (st != BZ_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    double* D = reinterpret_cast<double*>(static_cast<char*>(workspace) + pairdist_workspace(f));
    st = pairdist_on_device(voted, f, d, ld, D, workspace, s, true);
    if (st != BZ_OK) return st;
    st = bz_bulyan_select(D, f, c, selected, stream);
    if (st != BZ_OK) return st;
    if (d == 0) return BZ_OK;
    const int theta = f - 2 * c;
    return trimmed_mean_on_device(voted, d, ld, selected, theta, theta - 2 * c, out, s);
}

