// Pairwise squared distances between the f voted gradients - the O(f^2 d) part of the Krum family
// (Sec. 1.2; cost in Appendix A.1): the binary32 and binary64 kernels, the dispatch between them and the
// integer tensor-core kernel (pairdist_i8_kernel.cuh, the default for f = 25 and 49), and the entry point
// that keeps its scratch in a built-in array.
//
// The kernels here accumulate the difference form sum_j (v_a[j] - v_b[j])^2: its accuracy does not depend
// on a common offset of the rows (gradients share a large per-coordinate mean) nor on the size of an
// attacker's payload in other rows.  The binary32 kernels are bound by the FP32 pipe (f(f-1) add/fma
// lane-operations per coordinate) and serve the shapes the integer kernel does not take, and
// bz_pairdist_static.  The binary64 kernel (f = 25 and 49) answers where the integer kernel's error bound
// or a row's values ask for a recomputation, and for rows too short for that kernel.
#include <atomic>
#include <cstdlib>
#include <cstring>

#include "pairdist_tile.cuh"

namespace bz {

namespace {

// ------------------------------------------------------------------------------------------------
// Register-tiled kernel.  The F rows are split into NB = F/T residue classes; a thread owns one
// unordered pair of classes (bi <= bj), i.e. the T x T row pairs (bi + NB*t, bj + NB*u), and one of
// G interleaved coordinate groups of every tile.  A CTA streams tiles of kTD coordinates of all F
// rows through a double-buffered shared-memory stage (cp.async, 16 bytes per request).
// Sums: binary32 in registers over kFlush tiles (kFlush * kTD / G coordinates per thread), then
// the G groups of a pair are added in binary32 in a fixed order and the result goes into the CTA's
// binary64 accumulator in shared memory; one fixed-order reduction over CTAs finishes.
// The result is bit-reproducible from run to run.
// W bytes per request (16, 8 or 4: what the rows' alignment allows); bytes past src_bytes are filled with zeros
template <int W> __device__ __forceinline__ void cp_async_w(void* smem_dst, const void* gmem_src, int src_bytes) {
    const unsigned dst = static_cast<unsigned>(__cvta_generic_to_shared(smem_dst));
    if constexpr (W == 16)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(gmem_src), "r"(src_bytes));
    else if constexpr (W == 8)
        asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;\n" ::"r"(dst), "l"(gmem_src), "r"(src_bytes));
    else
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;\n" ::"r"(dst), "l"(gmem_src), "r"(src_bytes));
}
// One tile (kTD coordinates from j0, zeros past d) of F rows into dst[F][kRowStride], NT threads.
template <int F, int NT, int W>
__device__ __forceinline__ void stage_rows_w(float* dst, const float* __restrict__ v, int64_t d, int64_t ld, int64_t j0, int tid) {
    constexpr int E = W / 4, per_row = kTD / E;
    for (int idx = tid; idx < F * per_row; idx += NT) {
        const int row = idx / per_row, c = idx - row * per_row;
        const int64_t j = j0 + E * c;
        const int64_t left = d - j;
        const int bytes = left >= E ? W : (left > 0 ? static_cast<int>(left) * 4 : 0);
        const float* src = bytes ? v + row * ld + j : v;  // zero-byte requests still name a valid address
        cp_async_w<W>(dst + row * kRowStride + E * c, src, bytes);
    }
}
// width: the bytes per request the rows allow (uniform over the launch)
template <int F, int NT>
__device__ __forceinline__ void stage_rows(float* dst, const float* __restrict__ v, int64_t d, int64_t ld, int64_t j0, int tid, int width) {
    if (width == 16)
        stage_rows_w<F, NT, 16>(dst, v, d, ld, j0, tid);
    else if (width == 8)
        stage_rows_w<F, NT, 8>(dst, v, d, ld, j0, tid);
    else
        stage_rows_w<F, NT, 4>(dst, v, d, ld, j0, tid);
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

template <int F, int T, int G>
__global__ void __launch_bounds__(PairTile<F, T, G>::NT, tiled_ctas_per_sm<F, T, G>())
    pairdist_tiled_kernel(const float* __restrict__ v, int64_t d, int64_t ld, int width, double* __restrict__ partial,
                          const int* __restrict__ gate) {
    using PT = PairTile<F, T, G>;
    if (gate != nullptr && *gate == 0) return;  // the integer kernel's distances stand
    constexpr int NB = PT::NB, NPB = PT::NPB, NT = PT::NT, TT = PT::TT;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* stage0 = reinterpret_cast<float*>(smem_raw);                            // 2 x [F][kRowStride]
    float* red = stage0 + 2 * F * kRowStride;                                      // [G][NPB][TT]
    double* dsum = reinterpret_cast<double*>(red + NT * TT + ((NT * TT) & 1));     // [NPB][TT]

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
    for (int e = tid; e < NPB * TT; e += NT) dsum[e] = 0.0;

    const int64_t n_tiles = (d + kTD - 1) / kTD;
    auto load_tile = [&](int buf, int64_t tile) {
        stage_rows<F, NT>(stage0 + buf * F * kRowStride, v, d, ld, tile * kTD, tid, width);
        cp_async_commit();
    };

    float acc[TT];
#pragma unroll
    for (int e = 0; e < TT; ++e) acc[e] = 0.f;

    int64_t tile = blockIdx.x;
    int buf = 0, since_flush = 0;
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

        accumulate_tile<F, T, G>(stage0 + buf * F * kRowStride, bi, bj, g, acc);
        ++since_flush;
        if (since_flush == kFlush || next >= n_tiles) {  // uniform over the CTA
            since_flush = 0;
#pragma unroll
            for (int e = 0; e < TT; ++e) {
                red[tid * TT + e] = acc[e];  // tid = g * NPB + pb
                acc[e] = 0.f;
            }
            __syncthreads();
            for (int e = g; e < TT; e += G) {
                float s = 0.f;
#pragma unroll
                for (int g2 = 0; g2 < G; ++g2) s += red[(g2 * NPB + pb) * TT + e];
                dsum[pb * TT + e] += static_cast<double>(s);
            }
        }
        __syncthreads();
        buf ^= 1;
    }
    __syncthreads();
    double* mine = partial + static_cast<size_t>(blockIdx.x) * NPB * TT;
    for (int e = tid; e < NPB * TT; e += NT) mine[e] = dsum[e];
}

// ------------------------------------------------------------------------------------------------
// The same tiling in binary64: differences, squares and sums all in double precision, so the result is
// the oracle's up to a few units of 2^-53 per term - whatever the data.  This is the kernel that answers
// when the integer kernel's error bound does not fit the tolerance (it reads that flag and returns at once
// otherwise), and for rows too short for the integer kernel.  Bound by the FP64 pipe: one add and one
// multiply-add per pair and coordinate, about 2.5x the time of the binary32 kernel.
// Every thread keeps its T x T sums for its whole share of the tiles; the G coordinate groups of a pair
// are added in a fixed order at the end.  Partial sums have the layout of the binary32 kernel's.
template <int F, int T, int G> constexpr size_t f64_smem_bytes() {
    using PT = PairTile<F, T, G>;
    return size_t(2) * F * kRowStride * 4 + size_t(PT::NT) * PT::TT * 8;
}

template <int F, int T, int G>
__global__ void __launch_bounds__(PairTile<F, T, G>::NT, 1)
    pairdist_f64_kernel(const float* __restrict__ v, int64_t d, int64_t ld, int width, double* __restrict__ partial,
                        const int* __restrict__ gate) {
    using PT = PairTile<F, T, G>;
    if (gate != nullptr && *gate == 0) return;  // the integer kernel's distances stand
    constexpr int NB = PT::NB, NPB = PT::NPB, NT = PT::NT, TT = PT::TT;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* stage0 = reinterpret_cast<float*>(smem_raw);                              // 2 x [F][kRowStride]
    double* red = reinterpret_cast<double*>(stage0 + 2 * F * kRowStride);            // [G][NPB][TT]
    static_assert((2 * F * kRowStride * 4) % 8 == 0, "binary64 buffer alignment");

    const int tid = threadIdx.x;
    int bi, bj, g;
    pair_of_thread<F, T, G>(tid, bi, bj, g);
    const int pb = tid % NPB;

    const int64_t n_tiles = (d + kTD - 1) / kTD;
    auto load_tile = [&](int buf, int64_t tile) {
        stage_rows<F, NT>(stage0 + buf * F * kRowStride, v, d, ld, tile * kTD, tid, width);
        cp_async_commit();
    };

    double acc[TT];
#pragma unroll
    for (int e = 0; e < TT; ++e) acc[e] = 0.0;

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
        const float* base = stage0 + buf * F * kRowStride;
#pragma unroll 1
        for (int c = g; c < kTD; c += G) {
            double b[T];
#pragma unroll
            for (int u = 0; u < T; ++u) b[u] = static_cast<double>(base[(bj + NB * u) * kRowStride + c]);
#pragma unroll
            for (int t = 0; t < T; ++t) {
                const double a = static_cast<double>(base[(bi + NB * t) * kRowStride + c]);
#pragma unroll
                for (int u = 0; u < T; ++u) {
                    const double e = a - b[u];
                    acc[t * T + u] = fma(e, e, acc[t * T + u]);
                }
            }
        }
        __syncthreads();
        buf ^= 1;
    }
#pragma unroll
    for (int e = 0; e < TT; ++e) red[tid * TT + e] = acc[e];  // tid = g * NPB + pb
    __syncthreads();
    double* mine = partial + static_cast<size_t>(blockIdx.x) * NPB * TT;
    for (int e = g; e < TT; e += G) {
        double s = 0.0;
#pragma unroll
        for (int g2 = 0; g2 < G; ++g2) s += red[(g2 * NPB + pb) * TT + e];
        mine[pb * TT + e] = s;
    }
}

// ------------------------------------------------------------------------------------------------
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
// host side

int pairdist_ctas(int64_t d, int tile, int per_sm = 1) {
    int64_t n_tiles = (d + tile - 1) / tile;
    if (n_tiles > kNumSMs * per_sm) n_tiles = kNumSMs * per_sm;
    if (n_tiles < 1) n_tiles = 1;
    return static_cast<int>(n_tiles);
}

template <int F, int T, int G> constexpr size_t tiled_partial_doubles() {
    return static_cast<size_t>(kNumSMs) * tiled_ctas_per_sm<F, T, G>() * PairTile<F, T, G>::NPB * PairTile<F, T, G>::TT;
}

// bytes per staging request that every row start allows: 16, 8 or 4
inline int row_width(const float* v, int64_t ld) {
    const uintptr_t bits = reinterpret_cast<uintptr_t>(v) | static_cast<uintptr_t>(ld * 4);
    return bits % 16 == 0 ? 16 : (bits % 8 == 0 ? 8 : 4);
}

template <int F, int T, int G>
int launch_pairdist_tiled(const float* v, int64_t d, int64_t ld, double* dist, double* partial, const int* gate, cudaStream_t s) {
    constexpr int NT = PairTile<F, T, G>::NT;
    constexpr int smem = static_cast<int>(tiled_smem_bytes<F, T, G>());
    cudaError_t e = cudaFuncSetAttribute(pairdist_tiled_kernel<F, T, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return cuda_failed(e);
    const int ctas = pairdist_ctas(d, kTD, tiled_ctas_per_sm<F, T, G>());
    pairdist_tiled_kernel<F, T, G><<<ctas, NT, smem, s>>>(v, d, ld, row_width(v, ld), partial, gate);
    note_launch();
    int st = check_launch();
    if (st != BZ_OK) return st;
    pairdist_tiled_reduce_kernel<F, T, G><<<(F * F + 127) / 128, 128, 0, s>>>(partial, ctas, dist, gate);
    note_launch();
    return check_launch();
}

template <int F, int T, int G>
int launch_pairdist_f64(const float* v, int64_t d, int64_t ld, double* dist, double* partial, const int* gate, cudaStream_t s) {
    constexpr int NT = PairTile<F, T, G>::NT;
    constexpr int smem = static_cast<int>(f64_smem_bytes<F, T, G>());
    cudaError_t e = cudaFuncSetAttribute(pairdist_f64_kernel<F, T, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return cuda_failed(e);
    const int ctas = pairdist_ctas(d, kTD, 1);  // never more CTAs than the binary32 kernel's workspace provides for
    pairdist_f64_kernel<F, T, G><<<ctas, NT, smem, s>>>(v, d, ld, row_width(v, ld), partial, gate);
    note_launch();
    int st = check_launch();
    if (st != BZ_OK) return st;
    pairdist_tiled_reduce_kernel<F, T, G><<<(F * F + 127) / 128, 128, 0, s>>>(partial, ctas, dist, gate);
    note_launch();
    return check_launch();
}

// BZ_PAIRDIST_PATH=fp32 keeps the distances off the tensor cores and on the binary32 kernels; =fp64 on the
// binary64 kernel (where it exists); =i8 takes the integer kernel's result even where its error bound asks
// for the binary64 kernel (for tests of that kernel).
enum { kPathAuto = 0, kPathFp32 = 1, kPathI8 = 2, kPathFp64 = 3 };
int pairdist_path() {
    const char* e = std::getenv("BZ_PAIRDIST_PATH");
    if (e == nullptr) return kPathAuto;
    if (std::strcmp(e, "fp32") == 0) return kPathFp32;
    if (std::strcmp(e, "i8") == 0) return kPathI8;
    if (std::strcmp(e, "fp64") == 0) return kPathFp64;
    return kPathAuto;
}

}  // namespace

bool pairdist_i8_has(int f);                  // pairdist_i8.cu
size_t pairdist_i8_workspace(int f);
int pairdist_i8(const float* v, int f, int64_t d, int64_t ld, double* dist, void* ws, int* flag, int force, cudaStream_t s);

int pairdist_path_fp32_only() { return pairdist_path() == kPathFp32; }
int pairdist_path_i8_forced() { return pairdist_path() == kPathI8; }
int pairdist_path_fp64_only() { return pairdist_path() == kPathFp64; }

// the partial sums of the binary32 kernels alone (what bz_pairdist_static keeps in its array)
size_t pairdist_workspace_fp32(int f) {
    size_t doubles;
    if (f == 25)
        doubles = tiled_partial_doubles<BZ_PD_25>();
    else if (f == 49)
        doubles = tiled_partial_doubles<BZ_PD_49>();
    else
        doubles = static_cast<size_t>(kNumSMs) * f * (f - 1) / 2;
    if (doubles < 32) doubles = 32;
    return round_up(doubles * sizeof(double), 256);
}

// binary32 partial sums, the call's two status words (256 bytes), then the integer kernel's partial matrices
constexpr size_t kStatusBytes = 256;
size_t pairdist_workspace(int f) { return pairdist_workspace_fp32(f) + kStatusBytes + pairdist_i8_workspace(f); }
int* pairdist_status_words(void* ws, int f) { return reinterpret_cast<int*>(static_cast<char*>(ws) + pairdist_workspace_fp32(f)); }
void* pairdist_i8_part(void* ws, int f) { return static_cast<char*>(ws) + pairdist_workspace_fp32(f) + kStatusBytes; }
// a call on which the integer kernel does not run clears the status words
int pairdist_clear_status(void* ws, int f, cudaStream_t s) {
    const cudaError_t e = cudaMemsetAsync(pairdist_status_words(ws, f), 0, 2 * sizeof(int), s);
    return e == cudaSuccess ? BZ_OK : cuda_failed(e);
}

// The binary32 difference-form kernels.  gate != nullptr: they run only if *gate (device) is not 0.
int pairdist_fp32(const float* v, int f, int64_t d, int64_t ld, double* dist, double* partial, const int* gate, cudaStream_t s);

// The binary64 kernel exists for the shapes of the integer kernel, f = 25 or 49, rows on any 4-byte boundary.
bool pairdist_f64_has(const float* v, int f, int64_t ld) {
    (void)v;
    (void)ld;
    return f == 25 || f == 49;
}
int pairdist_f64(const float* v, int f, int64_t d, int64_t ld, double* dist, double* partial, const int* gate, cudaStream_t s) {
    if (gate == nullptr) note_path(BZ_PATH_FP64);
    if (f == 25) return launch_pairdist_f64<BZ_PD_25>(v, d, ld, dist, partial, gate, s);
    return launch_pairdist_f64<BZ_PD_49>(v, d, ld, dist, partial, gate, s);
}

// tensor_cores: the workspace has room for the status words and the integer kernel (pairdist_workspace, not _fp32)
int pairdist_on_device(const float* v, int f, int64_t d, int64_t ld, double* dist, void* ws, cudaStream_t s, bool tensor_cores) {
    double* partial = static_cast<double*>(ws);
    const int* gate = nullptr;
    const int path = pairdist_path();
    if (tensor_cores) {
        int* flag = pairdist_status_words(ws, f);
        int st = 1;
        if (path != kPathFp32 && path != kPathFp64) st = pairdist_i8(v, f, d, ld, dist, pairdist_i8_part(ws, f), flag, path == kPathI8, s);
        if (st == BZ_OK) {
            note_path(BZ_PATH_TENSOR);
            return pairdist_f64(v, f, d, ld, dist, partial, flag, s);  // runs only if the flag asks for it
        } else if (st == 1) {
            st = pairdist_clear_status(ws, f, s);
            if (st != BZ_OK) return st;
            // rows too short for the integer kernel: binary64 costs nothing there and keeps the tolerance
            if (path != kPathFp32 && d > 0 && pairdist_f64_has(v, f, ld)) return pairdist_f64(v, f, d, ld, dist, partial, nullptr, s);
        } else {
            return st;
        }
    }
    return pairdist_fp32(v, f, d, ld, dist, partial, gate, s);
}

int pairdist_fp32(const float* v, int f, int64_t d, int64_t ld, double* dist, double* partial, const int* gate, cudaStream_t s) {
    if (gate == nullptr) note_path(BZ_PATH_FP32);
    if (f == 25) return launch_pairdist_tiled<BZ_PD_25>(v, d, ld, dist, partial, gate, s);
    if (f == 49) return launch_pairdist_tiled<BZ_PD_49>(v, d, ld, dist, partial, gate, s);
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
    return pairdist_on_device(voted, f, d, ld, dist, workspace, static_cast<cudaStream_t>(stream), true);
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
// device address of the array on each device, once resolved.  Host threads may make a device's first call
// at the same time: they all store the same address, atomically.  cudaDeviceReset() invalidates the address
// (the next context maps the image anew); a process that resets a device must not call this entry point on
// it afterwards.
std::atomic<void*> g_static_scratch_addr[kMaxDevices];

// The array's name is only a handle on the host side; kernels need its device address, which the
// runtime hands out per device.
int static_scratch(void** ptr) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_failed(e);
    if (dev < 0 || dev >= kMaxDevices) return BZ_ERR_UNSUPPORTED;
    void* p = g_static_scratch_addr[dev].load(std::memory_order_acquire);
    if (p == nullptr) {
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return cuda_failed(e);
        if (p == nullptr || !aligned256(p)) return BZ_ERR_WORKSPACE;
        g_static_scratch_addr[dev].store(p, std::memory_order_release);
    }
    *ptr = p;
    return BZ_OK;
}

}  // namespace

extern "C" int bz_pairdist_static(const float* voted, int f, int64_t d, int64_t ld, double* dist, void* stream) {
    int st = validate_rows(voted, f, d, ld);
    if (st != BZ_OK) return st;
    if (dist == nullptr) return BZ_ERR_INVALID_ARG;
    if (pairdist_workspace_fp32(f) > kStaticScratchBytes) return BZ_ERR_STATIC_LIMIT;
    void* scratch = nullptr;
    st = static_scratch(&scratch);
    if (st != BZ_OK) return st;
    // Nothing in the array has to start at zero: the tiled kernel overwrites every partial sum the
    // reduction reads, and the generic kernel clears its own slots before it accumulates.
    return pairdist_on_device(voted, f, d, ld, dist, scratch, static_cast<cudaStream_t>(stream), false);
}
