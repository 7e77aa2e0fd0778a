// The Krum family on the f voted gradients: pairwise squared distances, Multi-Krum selection and
// mean, Bulyan's iterated selection and its trimmed mean around the median (Sec. 1.2, Sec. 6.1).
#include "bz_common.cuh"

namespace bz {

namespace {

// ------------------------------------------------------------------------------------------------
// Pairwise distances, register-tiled.  The f rows are split into NB = F/T residue classes; a thread
// owns one unordered pair of classes (bi <= bj), i.e. the T x T row pairs (bi + NB*t, bj + NB*t'),
// and one of G interleaved coordinate groups of every tile.  A CTA streams tiles of TD coordinates
// of all F rows through a double-buffered shared-memory stage (cp.async, 16 bytes per request).
// Sums: binary32 inside one tile (TD / G coordinates per thread), binary64 across tiles, then one
// fixed-order reduction over CTAs and groups - bit-reproducible from run to run.
template <int F, int T> struct PairTile {
    static constexpr int NB = F / T;
    static constexpr int NPB = NB * (NB + 1) / 2;
    static_assert(NB * T == F, "T must divide F");
};

constexpr int kTD = 256;        // coordinates per tile
constexpr int kRowPad = 4;      // floats; keeps the row stride an odd number of 16-byte units
constexpr int kRowStride = kTD + kRowPad;

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src, int src_bytes) {
    const unsigned dst = static_cast<unsigned>(__cvta_generic_to_shared(smem_dst));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(gmem_src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

template <int F, int T, int G>
__global__ void __launch_bounds__(PairTile<F, T>::NPB* G)
    pairdist_tiled_kernel(const float* __restrict__ v, int64_t d, int64_t ld, double* __restrict__ partial) {
    using PT = PairTile<F, T>;
    constexpr int NB = PT::NB, NPB = PT::NPB, NT = NPB * G;
    extern __shared__ __align__(16) float smem[];
    float* stage[2] = {smem, smem + F * kRowStride};

    const int tid = threadIdx.x;
    const int pb = tid % NPB, g = tid / NPB;
    int bi = 0, bj = 0;
    {
        int rest = pb;
        while (rest >= NB - bi) {
            rest -= NB - bi;
            ++bi;
        }
        bj = bi + rest;
    }

    const int64_t n_tiles = (d + kTD - 1) / kTD;
    auto load_tile = [&](int buf, int64_t tile) {
        const int64_t j0 = tile * kTD;
        constexpr int per_row = kTD / 4;
        for (int idx = tid; idx < F * per_row; idx += NT) {
            const int row = idx / per_row, c4 = idx - row * per_row;
            const int64_t j = j0 + 4 * c4;
            const int64_t left = d - j;
            const int bytes = left >= 4 ? 16 : (left > 0 ? static_cast<int>(left) * 4 : 0);
            const float* src = bytes ? v + row * ld + j : v;  // zero-byte requests still name a valid address
            cp_async16(stage[buf] + row * kRowStride + 4 * c4, src, bytes);
        }
        cp_async_commit();
    };

    double dacc[T * T];
#pragma unroll
    for (int e = 0; e < T * T; ++e) dacc[e] = 0.0;

    int64_t tile = blockIdx.x;
    int buf = 0;
    if (tile < n_tiles) load_tile(0, tile);
    for (; tile < n_tiles; tile += gridDim.x) {
        const int64_t next = tile + gridDim.x;
        if (next < n_tiles) {
            load_tile(buf ^ 1, next);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();

        float acc[T * T];
#pragma unroll
        for (int e = 0; e < T * T; ++e) acc[e] = 0.f;
        const float* base = stage[buf];
#pragma unroll 1
        for (int c4 = g; c4 < kTD / 4; c4 += G) {
            float4 a[T], b[T];
#pragma unroll
            for (int t = 0; t < T; ++t) {
                a[t] = *reinterpret_cast<const float4*>(base + (bi + NB * t) * kRowStride + 4 * c4);
                b[t] = *reinterpret_cast<const float4*>(base + (bj + NB * t) * kRowStride + 4 * c4);
            }
#pragma unroll
            for (int t = 0; t < T; ++t)
#pragma unroll
                for (int u = 0; u < T; ++u) {
                    float s = acc[t * T + u];
                    float e;
                    e = a[t].x - b[u].x; s = fmaf(e, e, s);
                    e = a[t].y - b[u].y; s = fmaf(e, e, s);
                    e = a[t].z - b[u].z; s = fmaf(e, e, s);
                    e = a[t].w - b[u].w; s = fmaf(e, e, s);
                    acc[t * T + u] = s;
                }
        }
#pragma unroll
        for (int e = 0; e < T * T; ++e) dacc[e] += static_cast<double>(acc[e]);
        __syncthreads();
        buf ^= 1;
    }
    double* mine = partial + (static_cast<size_t>(blockIdx.x) * NT + tid) * (T * T);
#pragma unroll
    for (int e = 0; e < T * T; ++e) mine[e] = dacc[e];
}

// dist[a][b] = sum over CTAs (ascending) and groups (ascending) of the owning thread's element
template <int F, int T, int G>
__global__ void pairdist_tiled_reduce_kernel(const double* __restrict__ partial, int n_ctas, double* __restrict__ dist) {
    using PT = PairTile<F, T>;
    constexpr int NB = PT::NB, NPB = PT::NPB, NT = NPB * G;
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
    for (int cta = 0; cta < n_ctas; ++cta)
        for (int g = 0; g < G; ++g) s += partial[(static_cast<size_t>(cta) * NT + g * NPB + pb) * (T * T) + t * T + u];
    dist[a * F + b] = s;
    dist[b * F + a] = s;
}

// Any f, any alignment: a CTA stages kGT coordinates of all rows with scalar loads; pair p is
// always summed by thread p % blockDim of the CTA, binary32 inside the stage, binary64 across.
constexpr int kGT = 64;
__global__ void __launch_bounds__(256)
    pairdist_generic_kernel(const float* __restrict__ v, int f, int64_t d, int64_t ld, double* __restrict__ partial) {
    __shared__ float tile[BZ_MAX_F][kGT + 1];
    const int n_pairs = f * (f - 1) / 2;
    double* mine = partial + static_cast<size_t>(blockIdx.x) * n_pairs;
    for (int p = threadIdx.x; p < n_pairs; p += blockDim.x) mine[p] = 0.0;
    const int64_t n_tiles = (d + kGT - 1) / kGT;
    for (int64_t tile_i = blockIdx.x; tile_i < n_tiles; tile_i += gridDim.x) {
        const int64_t j0 = tile_i * kGT;
        for (int idx = threadIdx.x; idx < f * kGT; idx += blockDim.x) {
            const int row = idx / kGT, c = idx % kGT;
            tile[row][c] = (j0 + c < d) ? v[row * ld + j0 + c] : 0.f;
        }
        __syncthreads();
        for (int p = threadIdx.x; p < n_pairs; p += blockDim.x) {
            // p -> (a, b), a < b, row-major over the strict upper triangle
            int a = 0, rest = p;
            while (rest >= f - 1 - a) {
                rest -= f - 1 - a;
                ++a;
            }
            const int b = a + 1 + rest;
            float s = 0.f;
            for (int c = 0; c < kGT; ++c) {
                const float e = tile[a][c] - tile[b][c];
                s = fmaf(e, e, s);
            }
            mine[p] += static_cast<double>(s);
        }
        __syncthreads();
    }
}

__global__ void pairdist_generic_reduce_kernel(const double* __restrict__ partial, int n_ctas, int f,
                                               double* __restrict__ dist) {
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p < f) dist[p * f + p] = 0.0;
    const int n_pairs = f * (f - 1) / 2;
    if (p >= n_pairs) return;
    int a = 0, rest = p;
    while (rest >= f - 1 - a) {
        rest -= f - 1 - a;
        ++a;
    }
    const int b = a + 1 + rest;
    double s = 0.0;
    for (int cta = 0; cta < n_ctas; ++cta) s += partial[static_cast<size_t>(cta) * n_pairs + p];
    dist[a * f + b] = s;
    dist[b * f + a] = s;
}

// ------------------------------------------------------------------------------------------------
// Selection kernels: one CTA, thread a owns row a.

// Krum score of row a inside the rows flagged in `active`: the nb smallest distances to the other
// active rows, added in ascending order.  (Insertion sort in local memory; f <= BZ_MAX_F.)
__device__ double krum_score_row(const double* dist, int f, const unsigned char* active, int a, int nb) {
    double buf[BZ_MAX_F];
    int n = 0;
    for (int b = 0; b < f; ++b) {
        if (b == a || !active[b]) continue;
        const double x = dist[a * f + b];
        int pos = n++;
        while (pos > 0 && buf[pos - 1] > x) {
            buf[pos] = buf[pos - 1];
            --pos;
        }
        buf[pos] = x;
    }
    double s = 0.0;
    for (int t = 0; t < nb; ++t) s += buf[t];
    return s;
}

__global__ void __launch_bounds__(BZ_MAX_F) krum_select_kernel(const double* __restrict__ dist, int f, int c, int m,
                                                               int32_t* __restrict__ selected) {
    __shared__ double score[BZ_MAX_F];
    __shared__ unsigned char active[BZ_MAX_F];
    const int a = threadIdx.x;
    if (a < f) active[a] = 1;
    __syncthreads();
    if (a < f) score[a] = krum_score_row(dist, f, active, a, f - c - 2);
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
    __syncthreads();
    const int theta = f - 2 * c;
    for (int t = 0; t < theta; ++t) {
        const int n = f - t;
        int nb = n - c - 2;
        if (nb < 1) nb = 1;
        if (nb > n - 1) nb = n - 1;
        if (a < f && active[a]) score[a] = (n > 1) ? krum_score_row(dist, f, active, a, nb) : 0.0;
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

// Window of the beta sorted values closest to the median: the greedy growth (lower neighbour on
// ties) is a merge of the two distance sequences, so a value's membership follows from its rank
// in that merge.  s[] ascending; returns the mean of the window (binary64 sum, ascending).
template <int THETA> __device__ __forceinline__ float window_mean(const float (&s)[THETA], int beta) {
    constexpr int MID = (THETA - 1) / 2;
    const float med = s[MID];
    float dist[THETA];
#pragma unroll
    for (int t = 0; t < THETA; ++t) dist[t] = fabsf(__fsub_rn(s[t], med));
    double sum = 0.0;
#pragma unroll
    for (int t = 0; t < THETA; ++t) {
        int rank;  // number of values taken before s[t]; the median itself is rank 0
        if (t == MID) {
            rank = 0;
        } else if (t < MID) {
            rank = MID - t;  // the median and the lower values nearer to it
#pragma unroll
            for (int u = MID + 1; u < THETA; ++u) rank += (dist[u] < dist[t]);
        } else {
            rank = t - MID;
#pragma unroll
            for (int u = 0; u < MID; ++u) rank += (dist[u] <= dist[t]);
        }
        if (rank < beta) sum += static_cast<double>(s[t]);
    }
    return static_cast<float>(sum / static_cast<double>(beta));
}

template <int THETA>
__global__ void __launch_bounds__(128) trimmed_mean_kernel(const float* __restrict__ v, int64_t d, int64_t ld,
                                                           const int32_t* __restrict__ selected, int beta,
                                                           float* __restrict__ out) {
    __shared__ int32_t sel[THETA];
    for (int t = threadIdx.x; t < THETA; t += blockDim.x) sel[t] = selected[t];
    __syncthreads();
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; j < d; j += stride) {
        int k[THETA];
#pragma unroll
        for (int t = 0; t < THETA; ++t) k[t] = order_key(__float_as_uint(__ldcs(v + sel[t] * ld + j)));
        SortNet<THETA>::run(k);
        float s[THETA];
#pragma unroll
        for (int t = 0; t < THETA; ++t) s[t] = __uint_as_float(key_bits(k[t]));
        out[j] = window_mean<THETA>(s, beta);
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
        const int mid = (theta - 1) / 2;
        const float med = __uint_as_float(key_bits(k[mid]));
        int lo = mid, hi = mid;
        while (hi - lo + 1 < beta) {
            const bool can_lo = lo > 0, can_hi = hi < theta - 1;
            bool take_lo = can_lo;
            if (can_lo && can_hi) {
                const float dl = fabsf(__fsub_rn(__uint_as_float(key_bits(k[lo - 1])), med));
                const float dh = fabsf(__fsub_rn(__uint_as_float(key_bits(k[hi + 1])), med));
                take_lo = dl <= dh;
            }
            if (take_lo) --lo; else ++hi;
        }
        double sum = 0.0;
        for (int t = lo; t <= hi; ++t) sum += static_cast<double>(__uint_as_float(key_bits(k[t])));
        out[j] = static_cast<float>(sum / static_cast<double>(beta));
    }
}

// ------------------------------------------------------------------------------------------------
// host side

int pairdist_ctas(int64_t d, int tile) {
    int64_t n_tiles = (d + tile - 1) / tile;
    if (n_tiles > kNumSMs) n_tiles = kNumSMs;
    if (n_tiles < 1) n_tiles = 1;
    return static_cast<int>(n_tiles);
}

template <int F, int T, int G> constexpr size_t tiled_partial_doubles() {
    return static_cast<size_t>(kNumSMs) * PairTile<F, T>::NPB * G * T * T;
}

size_t pairdist_workspace(int f) {
    size_t doubles;
    if (f == 25)
        doubles = tiled_partial_doubles<25, 5, 8>();
    else if (f == 49)
        doubles = tiled_partial_doubles<49, 7, 8>();
    else
        doubles = static_cast<size_t>(kNumSMs) * f * (f - 1) / 2;
    if (doubles < 32) doubles = 32;
    return round_up(doubles * sizeof(double), 256);
}

template <int F, int T, int G>
int launch_pairdist_tiled(const float* v, int64_t d, int64_t ld, double* dist, double* partial, cudaStream_t s) {
    constexpr int NT = PairTile<F, T>::NPB * G;
    constexpr int smem = 2 * F * kRowStride * static_cast<int>(sizeof(float));
    cudaError_t e = cudaFuncSetAttribute(pairdist_tiled_kernel<F, T, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return cuda_failed(e);
    const int ctas = pairdist_ctas(d, kTD);
    pairdist_tiled_kernel<F, T, G><<<ctas, NT, smem, s>>>(v, d, ld, partial);
    note_launch();
    int st = check_launch();
    if (st != BZ_OK) return st;
    pairdist_tiled_reduce_kernel<F, T, G><<<(F * F + 127) / 128, 128, 0, s>>>(partial, ctas, dist);
    note_launch();
    return check_launch();
}

int pairdist_on_device(const float* v, int f, int64_t d, int64_t ld, double* dist, void* ws, cudaStream_t s) {
    double* partial = static_cast<double*>(ws);
    const bool vec = aligned16(v) && (ld % 4 == 0);
    if (vec && f == 25) return launch_pairdist_tiled<25, 5, 8>(v, d, ld, dist, partial, s);
    if (vec && f == 49) return launch_pairdist_tiled<49, 7, 8>(v, d, ld, dist, partial, s);
    const int ctas = pairdist_ctas(d, kGT);
    pairdist_generic_kernel<<<ctas, 256, 0, s>>>(v, f, d, ld, partial);
    note_launch();
    int st = check_launch();
    if (st != BZ_OK) return st;
    const int n = f * f;  // covers both the pairs and the diagonal
    pairdist_generic_reduce_kernel<<<(n + 127) / 128, 128, 0, s>>>(partial, ctas, f, dist);
    note_launch();
    return check_launch();
}

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

template <int THETA>
int launch_trimmed(const float* v, int64_t d, int64_t ld, const int32_t* selected, int beta, float* out, cudaStream_t s) {
    int64_t grid = (d + 127) / 128;
    if (grid > kNumSMs * 16) grid = kNumSMs * 16;
    trimmed_mean_kernel<THETA><<<static_cast<int>(grid), 128, 0, s>>>(v, d, ld, selected, beta, out);
    note_launch();
    return check_launch();
}

int trimmed_mean_on_device(const float* v, int64_t d, int64_t ld, const int32_t* selected, int theta, int beta,
                           float* out, cudaStream_t s) {
    switch (theta) {
#define BZ_TM_CASE(N) \
    case N: return launch_trimmed<N>(v, d, ld, selected, beta, out, s);
        BZ_TM_CASE(5) BZ_TM_CASE(7) BZ_TM_CASE(9) BZ_TM_CASE(15) BZ_TM_CASE(17) BZ_TM_CASE(19) BZ_TM_CASE(21)
        BZ_TM_CASE(23) BZ_TM_CASE(25) BZ_TM_CASE(27) BZ_TM_CASE(29) BZ_TM_CASE(31) BZ_TM_CASE(33) BZ_TM_CASE(35)
        BZ_TM_CASE(37) BZ_TM_CASE(39) BZ_TM_CASE(41) BZ_TM_CASE(43) BZ_TM_CASE(45) BZ_TM_CASE(47) BZ_TM_CASE(49)
#undef BZ_TM_CASE
        default: break;
    }
    int64_t grid = (d + 127) / 128;
    if (grid > kNumSMs * 8) grid = kNumSMs * 8;
    trimmed_mean_generic_kernel<<<static_cast<int>(grid), 128, 0, s>>>(v, d, ld, selected, theta, beta, out);
    note_launch();
    return check_launch();
}

int validate_rows(const float* v, int f, int64_t d, int64_t ld) {
    if (d < 0 || f < 1 || (v == nullptr && d > 0)) return BZ_ERR_INVALID_ARG;  // an empty array may have no address
    if (f > BZ_MAX_F) return BZ_ERR_UNSUPPORTED;
    if (ld < d) return BZ_ERR_INVALID_ARG;
    return BZ_OK;
}

int check_workspace(void* ws, size_t have, size_t need) {
    if (ws == nullptr || !aligned256(ws) || have < need) return BZ_ERR_WORKSPACE;
    return BZ_OK;
}

}  // namespace

size_t krum_workspace_bytes(int op, int f) {
    const size_t pd = pairdist_workspace(f);
    if (op == BZ_OP_PAIRDIST) return pd;
    // multi-Krum / Bulyan: partial sums, then the f x f matrix
    return pd + round_up(static_cast<size_t>(f) * f * sizeof(double), 256);
}

}  // namespace bz

using namespace bz;

extern "C" int bz_pairdist(const float* voted, int f, int64_t d, int64_t ld, double* dist, void* workspace,
                           size_t workspace_bytes, void* stream) {
    int st = validate_rows(voted, f, d, ld);
    if (st != BZ_OK) return st;
    if (dist == nullptr) return BZ_ERR_INVALID_ARG;
    st = check_workspace(workspace, workspace_bytes, krum_workspace_bytes(BZ_OP_PAIRDIST, f));
    if (st != BZ_OK) return st;
    return pairdist_on_device(voted, f, d, ld, dist, workspace, static_cast<cudaStream_t>(stream));
}

extern "C" int bz_krum_select(const double* dist, int f, int c, int m, int32_t* selected, void* stream) {
    if (dist == nullptr || selected == nullptr || f < 1) return BZ_ERR_INVALID_ARG;
    if (f > BZ_MAX_F) return BZ_ERR_UNSUPPORTED;
    if (c < 0 || f < 2 * c + 3 || m < 1 || m > f) return BZ_ERR_PRECONDITION;
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
    st = pairdist_on_device(voted, f, d, ld, D, workspace, s);
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
    st = pairdist_on_device(voted, f, d, ld, D, workspace, s);
    if (st != BZ_OK) return st;
    st = bz_bulyan_select(D, f, c, selected, stream);
    if (st != BZ_OK) return st;
    if (d == 0) return BZ_OK;
    const int theta = f - 2 * c;
    return trimmed_mean_on_device(voted, d, ld, selected, theta, theta - 2 * c, out, s);
}

// ------------------------------------------------------------------------------------------------
// Pairwise distances without a caller workspace.
//
// Some hosts of this library may not allocate device memory at the moment they need the distance
// matrix: an operator plugged into a framework whose memory plan is frozen before the run, a
// serving or training loop that must not take the implicit device synchronisation an allocation
// can bring, a process confined to a fixed memory budget on a shared GPU.  For them the partial
// sums that bz_pairdist keeps in the caller's workspace live in the array below, which every GPU
// that loads the library holds from load to exit.
namespace {

constexpr size_t kStaticScratchBytes = BZ_STATIC_SCRATCH_BYTES;  // 4 MiB
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_static_scratch_addr[kMaxDevices] = {};  // device address of the array on each device, once resolved

// The array's name is only a handle on the host side; kernels need its device address, which the
// runtime hands out per device.
int static_scratch(void** ptr) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_failed(e);
    if (dev < 0 || dev >= kMaxDevices) return BZ_ERR_UNSUPPORTED;
    if (g_static_scratch_addr[dev] == nullptr) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return cuda_failed(e);
        if (p == nullptr || !aligned256(p)) return BZ_ERR_WORKSPACE;
        g_static_scratch_addr[dev] = p;
    }
    *ptr = g_static_scratch_addr[dev];
    return BZ_OK;
}

}  // namespace

extern "C" int bz_pairdist_static(const float* voted, int f, int64_t d, int64_t ld, double* dist, void* stream) {
    int st = validate_rows(voted, f, d, ld);
    if (st != BZ_OK) return st;
    if (dist == nullptr) return BZ_ERR_INVALID_ARG;
    if (krum_workspace_bytes(BZ_OP_PAIRDIST, f) > kStaticScratchBytes) return BZ_ERR_STATIC_LIMIT;
    void* scratch = nullptr;
    st = static_scratch(&scratch);
    if (st != BZ_OK) return st;
    // Nothing in the array has to start at zero: the tiled kernel overwrites every partial sum the
    // reduction reads, and the generic kernel clears its own slots before it accumulates.
    return pairdist_on_device(voted, f, d, ld, dist, scratch, static_cast<cudaStream_t>(stream));
}
