// Majority vote (Eq. 3), coordinate-wise median, and the two fused in one pass over the replicas.
//
// Register path: every thread owns VEC consecutive coordinates (VEC = 4 with 128-bit loads, 1 on the
// scalar path), streams the r copies of each of the f files once, votes them on their bit
// patterns, keeps the f winners as order keys in registers and selects the median with a
// comparator network.  HBM traffic is the algorithmic minimum: 4*r*f bytes in, 4 bytes out per
// coordinate.
#include <cstdlib>
#include <cstring>

#include "bz_common.cuh"

namespace bz {

// vote_median_tma.cu: BZ_OK / error, or 1 when the staged path does not apply
int vote_tma(const float* rep, int r, int f, int64_t d, int64_t ld_file, int64_t ld_rep, float* voted, int64_t ld_voted,
             cudaStream_t s);
int vote_median_tma(const float* rep, int r, int f, int64_t d, int64_t ld_file, int64_t ld_rep, float* out,
                    const ModelUpdate& upd, cudaStream_t s);

namespace {

constexpr int kBlock = 128;
constexpr ModelUpdate kNoUpdate = {nullptr, nullptr, 0.f, 0.f};

// BZ_VOTE_MEDIAN_PATH=registers keeps the fused pass on the register path (for profiling the two
// against each other); anything else lets the TMA-staged path run where it applies.
bool staged_path_enabled() {
    static const bool on = [] {
        const char* v = std::getenv("BZ_VOTE_MEDIAN_PATH");
        return !(v != nullptr && std::strcmp(v, "registers") == 0);
    }();
    return on;
}

// The vote alone through the fused kernel's bulk-copy ring: the loads do not care how the rows sit relative to
// 128-byte lines, and the winners leave as 128-bit stores from the stage (32-bit ones where the output is not
// 16-byte aligned).  Measured against the register kernel at d = 11.2 M: r = 3, f = 49 1.05 against 0.98 of the copy
// rate (rows off 128-byte lines: 1.00 against 0.86), r = 5 0.99 against 0.96, r = 7 0.89 against 0.78 - so it is the
// default wherever it applies.  BZ_VOTE_PATH=registers / =staged forces one or the other (read at every call).
bool vote_staged_enabled() {
    const char* v = std::getenv("BZ_VOTE_PATH");
    return !(v != nullptr && std::strcmp(v, "registers") == 0);
}

template <typename V> struct Lanes;
template <> struct Lanes<uint4> {
    static constexpr int n = 4;
    __device__ __forceinline__ static uint32_t get(const uint4& v, int c) {
        return c == 0 ? v.x : (c == 1 ? v.y : (c == 2 ? v.z : v.w));
    }
    __device__ __forceinline__ static uint4 make(const uint32_t (&a)[4]) { return make_uint4(a[0], a[1], a[2], a[3]); }
    __device__ __forceinline__ static void update(const ModelUpdate& u, int64_t j, const uint4& g) { apply_update4(u, j, g); }
};
template <> struct Lanes<uint2> {
    static constexpr int n = 2;
    __device__ __forceinline__ static uint32_t get(const uint2& v, int c) { return c == 0 ? v.x : v.y; }
    __device__ __forceinline__ static uint2 make(const uint32_t (&a)[2]) { return make_uint2(a[0], a[1]); }
    __device__ __forceinline__ static void update(const ModelUpdate& u, int64_t j, const uint2& g) {
        apply_update(u, 2 * j, __uint_as_float(g.x));
        apply_update(u, 2 * j + 1, __uint_as_float(g.y));
    }
};
template <> struct Lanes<uint32_t> {
    static constexpr int n = 1;
    __device__ __forceinline__ static uint32_t get(const uint32_t& v, int) { return v; }
    __device__ __forceinline__ static uint32_t make(const uint32_t (&a)[1]) { return a[0]; }
    __device__ __forceinline__ static void update(const ModelUpdate& u, int64_t j, uint32_t g) {
        apply_update(u, j, __uint_as_float(g));
    }
};

// the same update for coordinates n and up
ModelUpdate shifted(const ModelUpdate& u, int64_t n) {
    ModelUpdate t = u;
    if (t.w != nullptr) t.w += n;
    if (t.v != nullptr) t.v += n;
    return t;
}

// files fetched together before their votes are taken: keeps about 12 wide loads in flight
template <int R, int VEC> constexpr int files_per_batch() {
    constexpr int target_regs = 48;
    int b = target_regs / (R * VEC);
    return b < 1 ? 1 : b;
}

// n = number of V-wide coordinate groups; ld_file / ld_rep in units of V.  out may be null when
// only the model update is wanted.
template <int R, int F, typename V>
__global__ void __launch_bounds__(kBlock) vote_median_kernel(const V* __restrict__ rep, int64_t n, int64_t ld_file,
                                                              int64_t ld_rep, V* __restrict__ out, const ModelUpdate upd) {
    constexpr int VEC = Lanes<V>::n;
    constexpr int B = files_per_batch<R, VEC>();
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kBlock;
    for (int64_t j = static_cast<int64_t>(blockIdx.x) * kBlock + threadIdx.x; j < n; j += stride) {
        int key[VEC][F];
        const V* p = rep + j;
#pragma unroll
        for (int i0 = 0; i0 < F; i0 += B) {
            V x[B][R];
#pragma unroll
            for (int b = 0; b < B; ++b)
#pragma unroll
                for (int k = 0; k < R; ++k)
                    if (i0 + b < F) x[b][k] = ld_stream(p + k * ld_rep + (i0 + b) * ld_file);
#pragma unroll
            for (int b = 0; b < B; ++b)
                if (i0 + b < F) {
#pragma unroll
                    for (int c = 0; c < VEC; ++c) {
                        uint32_t copies[R];
#pragma unroll
                        for (int k = 0; k < R; ++k) copies[k] = Lanes<V>::get(x[b][k], c);
                        key[c][i0 + b] = order_key(vote_bits<R>(copies));
                    }
                }
        }
        uint32_t res[VEC];
#pragma unroll
        for (int c = 0; c < VEC; ++c) res[c] = key_bits(MedianNet<F>::run(key[c]));
        const V packed = Lanes<V>::make(res);
        if (out != nullptr) out[j] = packed;
        if (upd.w != nullptr) Lanes<V>::update(upd, j, packed);
    }
}

// grid.y = file, grid.x strides over coordinate groups.  gate != nullptr: the kernel runs only if *gate is
// not 0 (the repair of voted rows after a single-pass kernel that stopped early).
template <int R, typename V>
__global__ void __launch_bounds__(256) vote_kernel(const V* __restrict__ rep, int64_t n, int64_t ld_file,
                                                   int64_t ld_rep, V* __restrict__ voted, int64_t ld_voted,
                                                   const int* __restrict__ gate) {
    if (gate != nullptr && *gate == 0) return;
    constexpr int VEC = Lanes<V>::n;
    // coordinate groups per thread and trip: ~192 bytes of loads in flight whatever the width of a load
    constexpr int U = (12 * 4 / VEC / R) < 1 ? 1 : (12 * 4 / VEC / R);
    const int i = blockIdx.y;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    const V* src = rep + i * ld_file;
    V* dst = voted + i * ld_voted;
    for (int64_t j0 = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; j0 < n; j0 += stride * U) {
        V x[U][R];
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
            for (int k = 0; k < R; ++k)
                if (j0 + u * stride < n) x[u][k] = ld_stream(src + k * ld_rep + j0 + u * stride);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (j0 + u * stride >= n) break;
            uint32_t res[VEC];
#pragma unroll
            for (int c = 0; c < VEC; ++c) {
                uint32_t copies[R];
#pragma unroll
                for (int k = 0; k < R; ++k) copies[k] = Lanes<V>::get(x[u][k], c);
                res[c] = vote_bits<R>(copies);
            }
            dst[j0 + u * stride] = Lanes<V>::make(res);
        }
    }
}

// Any (r, f) within the limits, one coordinate per thread, arrays in local memory.  mode 0: vote
// only (writes voted), mode 1: vote + median (writes out).
__global__ void __launch_bounds__(128) generic_kernel(const uint32_t* __restrict__ rep, int r, int f, int64_t d,
                                                      int64_t ld_file, int64_t ld_rep, uint32_t* __restrict__ voted,
                                                      int64_t ld_voted, float* __restrict__ out, int mode,
                                                      const ModelUpdate upd) {
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; j < d; j += stride) {
        int key[BZ_MAX_F];
        for (int i = 0; i < f; ++i) {
            uint32_t x[BZ_MAX_R];
            for (int k = 0; k < r; ++k) x[k] = rep[k * ld_rep + i * ld_file + j];
            const uint32_t w = vote_bits_dyn(x, r);
            if (mode == 0)
                voted[i * ld_voted + j] = w;
            else
                key[i] = order_key(w);
        }
        if (mode == 0) continue;
        // element(s) of the wanted rank by counting, ties ordered by position
        const int want_hi = f / 2, want_lo = (f - 1) / 2;
        int k_lo = 0, k_hi = 0;
        for (int i = 0; i < f; ++i) {
            int rank = 0;
            for (int t = 0; t < f; ++t) rank += (key[t] < key[i]) || (key[t] == key[i] && t < i);
            if (rank == want_lo) k_lo = key[i];
            if (rank == want_hi) k_hi = key[i];
        }
        const float med = (f & 1) ? __uint_as_float(key_bits(k_lo))
                                  : __fadd_rn(__fmul_rn(0.5f, __uint_as_float(key_bits(k_lo))),
                                              __fmul_rn(0.5f, __uint_as_float(key_bits(k_hi))));
        if (out != nullptr) out[j] = med;
        if (upd.w != nullptr) apply_update(upd, j, med);
    }
}

int grid_for(int64_t work_items, int block, int ctas_per_sm) {
    int64_t need = (work_items + block - 1) / block;
    const int64_t cap = static_cast<int64_t>(kNumSMs) * ctas_per_sm;
    if (need > cap) need = cap;
    if (need < 1) need = 1;
    return static_cast<int>(need);
}

template <int R, int F, typename V>
int launch_vm(const float* rep, int64_t n, int64_t ld_file, int64_t ld_rep, float* out, const ModelUpdate& upd,
              cudaStream_t s) {
    if (n <= 0) return BZ_OK;
    constexpr int VEC = Lanes<V>::n;
    vote_median_kernel<R, F, V><<<grid_for(n, kBlock, 16), kBlock, 0, s>>>(
        reinterpret_cast<const V*>(rep), n, ld_file / VEC, ld_rep / VEC, reinterpret_cast<V*>(out), upd);
    note_launch();
    return check_launch();
}

// vec = coordinates per load the arrays' alignment allows: 4 (128-bit loads), 2 (64-bit) or 1; whatever is left
// past the last full group goes through the scalar kernel
template <int R, int F>
int vm_dispatch_vec(const float* rep, int64_t d, int64_t ld_file, int64_t ld_rep, float* out, const ModelUpdate& upd,
                    int vec, cudaStream_t s) {
    if (vec == 1) return launch_vm<R, F, uint32_t>(rep, d, ld_file, ld_rep, out, upd, s);
    const int64_t nv = d / vec;
    int st = vec == 4 ? launch_vm<R, F, uint4>(rep, nv, ld_file, ld_rep, out, upd, s)
                      : launch_vm<R, F, uint2>(rep, nv, ld_file, ld_rep, out, upd, s);
    if (st != BZ_OK) return st;
    return launch_vm<R, F, uint32_t>(rep + vec * nv, d - vec * nv, ld_file, ld_rep, out != nullptr ? out + vec * nv : nullptr,
                                     shifted(upd, vec * nv), s);
}

template <int R>
int vm_dispatch_f(const float* rep, int f, int64_t d, int64_t ld_file, int64_t ld_rep, float* out,
                  const ModelUpdate& upd, int vec, cudaStream_t s) {
    switch (f) {
        case 25: return vm_dispatch_vec<R, 25>(rep, d, ld_file, ld_rep, out, upd, vec, s);
        case 49: return vm_dispatch_vec<R, 49>(rep, d, ld_file, ld_rep, out, upd, vec, s);
        default: return 1;  // not specialised
    }
}

int launch_generic(const float* rep, int r, int f, int64_t d, int64_t ld_file, int64_t ld_rep, float* voted,
                   int64_t ld_voted, float* out, int mode, const ModelUpdate& upd, cudaStream_t s) {
    generic_kernel<<<grid_for(d, 128, 8), 128, 0, s>>>(reinterpret_cast<const uint32_t*>(rep), r, f, d, ld_file, ld_rep,
                                                       reinterpret_cast<uint32_t*>(voted), ld_voted, out, mode, upd);
    note_launch();
    return check_launch();
}

template <int R, typename V>
int launch_vote(const float* rep, int f, int64_t n, int64_t ld_file, int64_t ld_rep, float* voted, int64_t ld_voted,
                const int* gate, cudaStream_t s) {
    if (n <= 0) return BZ_OK;
    constexpr int VEC = Lanes<V>::n;
    // about 8 CTAs per SM over the whole (coordinate group, file) grid
    int64_t gx = (n + 255) / 256;
    const int64_t cap = (static_cast<int64_t>(kNumSMs) * 8 + f - 1) / f;
    if (gx > cap) gx = cap;
    if (gx < 1) gx = 1;
    dim3 grid(static_cast<unsigned>(gx), f);
    vote_kernel<R, V><<<grid, 256, 0, s>>>(reinterpret_cast<const V*>(rep), n, ld_file / VEC, ld_rep / VEC,
                                           reinterpret_cast<V*>(voted), ld_voted / VEC, gate);
    note_launch();
    return check_launch();
}

template <int R>
int vote_dispatch(const float* rep, int f, int64_t d, int64_t ld_file, int64_t ld_rep, float* voted, int64_t ld_voted,
                  int vec, cudaStream_t s, const int* gate = nullptr) {
    if (vec == 1) return launch_vote<R, uint32_t>(rep, f, d, ld_file, ld_rep, voted, ld_voted, gate, s);
    const int64_t nv = d / vec;
    int st = vec == 4 ? launch_vote<R, uint4>(rep, f, nv, ld_file, ld_rep, voted, ld_voted, gate, s)
                      : launch_vote<R, uint2>(rep, f, nv, ld_file, ld_rep, voted, ld_voted, gate, s);
    if (st != BZ_OK) return st;
    return launch_vote<R, uint32_t>(rep + vec * nv, f, d - vec * nv, ld_file, ld_rep, voted + vec * nv, ld_voted, gate, s);
}

// ------------------------------------------------------------------------------------------------
// The same kernels for copies that do not sit in one strided array: `rows` is a device table of r*f
// pointers, entry k*f + i = copy k of file i (d floats).  This is the layout of a parameter server
// that keeps what each worker sent in that worker's own buffer (K buffers of l gradients, Algorithm 1).
// Whether 128-bit loads may be used is decided on the device from the pointers themselves: the
// vector kernel returns at once unless every row (and the output) is 16-byte aligned, and the scalar
// kernel then takes either the tail or everything.
__device__ __forceinline__ bool rows_aligned(const float* const* rows, int count, bool out_aligned) {
    int ok = out_aligned ? 1 : 0;
    for (int t = threadIdx.x; t < count; t += blockDim.x) ok &= (reinterpret_cast<uintptr_t>(rows[t]) & 15u) == 0;
    return __syncthreads_and(ok) != 0;
}

template <int R, int F, typename V>
__global__ void __launch_bounds__(kBlock) vote_median_rows_kernel(const float* const* __restrict__ rows, int64_t d,
                                                                   float* __restrict__ out, int out_aligned) {
    constexpr int VEC = Lanes<V>::n;
    constexpr int B = files_per_batch<R, VEC>();
    __shared__ const float* tab[R * F];
    for (int t = threadIdx.x; t < R * F; t += kBlock) tab[t] = rows[t];
    const bool aligned = rows_aligned(rows, R * F, out_aligned != 0);   // contains the barrier that publishes tab
    int64_t begin, end;
    if (VEC == 4) {
        if (!aligned) return;
        begin = 0;
        end = d / 4;
    } else {
        begin = aligned ? (d / 4) * 4 : 0;
        end = d;
    }
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kBlock;
    for (int64_t j = begin + static_cast<int64_t>(blockIdx.x) * kBlock + threadIdx.x; j < end; j += stride) {
        int key[VEC][F];
#pragma unroll
        for (int i0 = 0; i0 < F; i0 += B) {
            V x[B][R];
#pragma unroll
            for (int b = 0; b < B; ++b)
#pragma unroll
                for (int k = 0; k < R; ++k)
                    if (i0 + b < F) x[b][k] = ld_stream(reinterpret_cast<const V*>(tab[k * F + i0 + b]) + j);
#pragma unroll
            for (int b = 0; b < B; ++b)
                if (i0 + b < F) {
#pragma unroll
                    for (int c = 0; c < VEC; ++c) {
                        uint32_t copies[R];
#pragma unroll
                        for (int k = 0; k < R; ++k) copies[k] = Lanes<V>::get(x[b][k], c);
                        key[c][i0 + b] = order_key(vote_bits<R>(copies));
                    }
                }
        }
        uint32_t res[VEC];
#pragma unroll
        for (int c = 0; c < VEC; ++c) res[c] = key_bits(MedianNet<F>::run(key[c]));
        reinterpret_cast<V*>(out)[j] = Lanes<V>::make(res);
    }
}

// Any (r, f) within the limits and any alignment.  mode 0: vote only (writes voted), mode 1: vote + median.
__global__ void __launch_bounds__(128) generic_rows_kernel(const float* const* __restrict__ rows, int r, int f, int64_t d,
                                                           uint32_t* __restrict__ voted, int64_t ld_voted,
                                                           float* __restrict__ out, int mode) {
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; j < d; j += stride) {
        int key[BZ_MAX_F];
        for (int i = 0; i < f; ++i) {
            uint32_t x[BZ_MAX_R];
            for (int k = 0; k < r; ++k) x[k] = reinterpret_cast<const uint32_t*>(rows[k * f + i])[j];
            const uint32_t w = vote_bits_dyn(x, r);
            if (mode == 0)
                voted[i * ld_voted + j] = w;
            else
                key[i] = order_key(w);
        }
        if (mode == 0) continue;
        const int want_hi = f / 2, want_lo = (f - 1) / 2;
        int k_lo = 0, k_hi = 0;
        for (int i = 0; i < f; ++i) {
            int rank = 0;
            for (int t = 0; t < f; ++t) rank += (key[t] < key[i]) || (key[t] == key[i] && t < i);
            if (rank == want_lo) k_lo = key[i];
            if (rank == want_hi) k_hi = key[i];
        }
        out[j] = (f & 1) ? __uint_as_float(key_bits(k_lo))
                         : __fadd_rn(__fmul_rn(0.5f, __uint_as_float(key_bits(k_lo))), __fmul_rn(0.5f, __uint_as_float(key_bits(k_hi))));
    }
}

template <int R, int F>
int launch_vm_rows(const float* const* rows, int64_t d, float* out, cudaStream_t s) {
    const int out_aligned = aligned16(out) ? 1 : 0;
    if (d >= 4) {
        vote_median_rows_kernel<R, F, uint4><<<grid_for(d / 4, kBlock, 16), kBlock, 0, s>>>(rows, d, out, out_aligned);
        note_launch();
        const int st = check_launch();
        if (st != BZ_OK) return st;
    }
    // the tail if the rows are aligned (at most 3 coordinates), everything otherwise: sized for the latter
    vote_median_rows_kernel<R, F, uint32_t><<<grid_for(d, kBlock, 16), kBlock, 0, s>>>(rows, d, out, out_aligned);
    note_launch();
    return check_launch();
}

template <int R>
int vm_rows_dispatch_f(const float* const* rows, int f, int64_t d, float* out, cudaStream_t s) {
    switch (f) {
        case 25: return launch_vm_rows<R, 25>(rows, d, out, s);
        case 49: return launch_vm_rows<R, 49>(rows, d, out, s);
        default: return 1;
    }
}

int validate_replicas(const float* rep, int r, int f, int64_t d, int64_t ld_file, int64_t ld_rep) {
    if (d < 0 || r < 1 || f < 1 || (r % 2) == 0) return BZ_ERR_INVALID_ARG;
    if (rep == nullptr && d > 0) return BZ_ERR_INVALID_ARG;  // an empty array may have no address
    if (r > BZ_MAX_R || f > BZ_MAX_F) return BZ_ERR_UNSUPPORTED;
    if (ld_file < d) return BZ_ERR_INVALID_ARG;
    if (r > 1 && ld_rep < d) return BZ_ERR_INVALID_ARG;
    return BZ_OK;
}

}  // namespace

// out may be null when upd.w is not: then only the updated state is written.
int vote_median_on_device(const float* rep, int r, int f, int64_t d, int64_t ld_file, int64_t ld_rep, float* out,
                          const ModelUpdate& upd, cudaStream_t s) {
    int vec = 1;
    if (aligned16(rep) && aligned16(out) && aligned16(upd.w) && aligned16(upd.v) && (ld_file % 4 == 0) && (r == 1 || ld_rep % 4 == 0))
        vec = 4;
    else if (aligned8(rep) && aligned8(out) && aligned8(upd.w) && aligned8(upd.v) && (ld_file % 2 == 0) && (r == 1 || ld_rep % 2 == 0))
        vec = 2;
    int st = 1;
    if (staged_path_enabled()) {
        st = vote_median_tma(rep, r, f, d, ld_file, ld_rep, out, upd, s);
        if (st != 1) {
            note_path(BZ_PATH_STAGED);
            return st;
        }
    }
    note_path(BZ_PATH_REGISTERS);
    switch (r) {
        case 1: st = vm_dispatch_f<1>(rep, f, d, ld_file, ld_rep, out, upd, vec, s); break;
        case 3: st = vm_dispatch_f<3>(rep, f, d, ld_file, ld_rep, out, upd, vec, s); break;
        case 5: st = vm_dispatch_f<5>(rep, f, d, ld_file, ld_rep, out, upd, vec, s); break;
        case 7: st = vm_dispatch_f<7>(rep, f, d, ld_file, ld_rep, out, upd, vec, s); break;
        default: break;
    }
    if (st == 1) {
        note_path(BZ_PATH_GENERIC);
        st = launch_generic(rep, r, f, d, ld_file, ld_rep, nullptr, 0, out, 1, upd, s);
    }
    return st;
}

}  // namespace bz

using namespace bz;

extern "C" int bz_vote_median(const float* replicas, int r, int f, int64_t d, int64_t ld_file, int64_t ld_replica,
                              float* out, void* stream) {
    int st = validate_replicas(replicas, r, f, d, ld_file, ld_replica);
    if (st != BZ_OK) return st;
    if (out == nullptr && d > 0) return BZ_ERR_INVALID_ARG;
    if (d == 0) return BZ_OK;
    return vote_median_on_device(replicas, r, f, d, ld_file, ld_replica, out, kNoUpdate, static_cast<cudaStream_t>(stream));
}

extern "C" int bz_median(const float* voted, int f, int64_t d, int64_t ld, float* out, void* stream) {
    int st = validate_replicas(voted, 1, f, d, ld, 0);
    if (st != BZ_OK) return st;
    if (out == nullptr && d > 0) return BZ_ERR_INVALID_ARG;
    if (d == 0) return BZ_OK;
    return vote_median_on_device(voted, 1, f, d, ld, 0, out, kNoUpdate, static_cast<cudaStream_t>(stream));
}

extern "C" int bz_vote(const float* replicas, int r, int f, int64_t d, int64_t ld_file, int64_t ld_replica,
                       float* voted, int64_t ld_voted, void* stream) {
    int st = validate_replicas(replicas, r, f, d, ld_file, ld_replica);
    if (st != BZ_OK) return st;
    if ((voted == nullptr && d > 0) || ld_voted < d) return BZ_ERR_INVALID_ARG;
    if (d == 0) return BZ_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // (small inputs stay on the register kernel unless asked: below ~100 MB of replicas the call is bound by its
    // launch, and the staged kernel adds a descriptor and a ring to that - 27 -> 46 us at d = 100 000)
    const bool asked = std::getenv("BZ_VOTE_PATH") != nullptr;
    const bool large = static_cast<double>(r) * f * static_cast<double>(d) * 4.0 >= 128.0 * 1024 * 1024;
    if (r > 1 && vote_staged_enabled() && (large || asked)) {
        st = vote_tma(replicas, r, f, d, ld_file, ld_replica, voted, ld_voted, s);
        if (st != 1) {
            if (st == BZ_OK) note_path(BZ_PATH_STAGED);
            return st;
        }
    }
    int vec = 1;
    if (aligned16(replicas) && aligned16(voted) && (ld_file % 4 == 0) && (ld_voted % 4 == 0) && (r == 1 || ld_replica % 4 == 0))
        vec = 4;
    else if (aligned8(replicas) && aligned8(voted) && (ld_file % 2 == 0) && (ld_voted % 2 == 0) && (r == 1 || ld_replica % 2 == 0))
        vec = 2;
    note_path(r == 1 || r == 3 || r == 5 || r == 7 ? BZ_PATH_REGISTERS : BZ_PATH_GENERIC);
    switch (r) {
        case 1: return vote_dispatch<1>(replicas, f, d, ld_file, ld_replica, voted, ld_voted, vec, s);
        case 3: return vote_dispatch<3>(replicas, f, d, ld_file, ld_replica, voted, ld_voted, vec, s);
        case 5: return vote_dispatch<5>(replicas, f, d, ld_file, ld_replica, voted, ld_voted, vec, s);
        case 7: return vote_dispatch<7>(replicas, f, d, ld_file, ld_replica, voted, ld_voted, vec, s);
        default: return launch_generic(replicas, r, f, d, ld_file, ld_replica, voted, ld_voted, nullptr, 0, kNoUpdate, s);
    }
}

namespace bz {
// bz_vote on the device's say-so: the vote kernels are enqueued and return at once unless *gate (device) is
// not 0.  Only for arrays the 128-bit kernels accept and r in {3, 5, 7} (the shapes of the single-pass kernels).
int vote_if(const float* replicas, int r, int f, int64_t d, int64_t ld_file, int64_t ld_replica, float* voted,
            int64_t ld_voted, const int* gate, cudaStream_t s) {
    switch (r) {
        case 3: return vote_dispatch<3>(replicas, f, d, ld_file, ld_replica, voted, ld_voted, 4, s, gate);
        case 5: return vote_dispatch<5>(replicas, f, d, ld_file, ld_replica, voted, ld_voted, 4, s, gate);
        case 7: return vote_dispatch<7>(replicas, f, d, ld_file, ld_replica, voted, ld_voted, 4, s, gate);
        default: return BZ_ERR_UNSUPPORTED;
    }
}
}  // namespace bz

extern "C" int bz_vote_median_host(const float* replicas_host, int r, int f, int64_t d, float* out_host,
                                   void* workspace, size_t workspace_bytes, void* stream) {
    int st = validate_replicas(replicas_host, r, f, d, d, static_cast<int64_t>(f) * d);
    if (st != BZ_OK) return st;
    if (out_host == nullptr && d > 0) return BZ_ERR_INVALID_ARG;
    if (d == 0) return BZ_OK;
    if (workspace == nullptr || !aligned256(workspace)) return BZ_ERR_WORKSPACE;
    if (workspace_bytes < bz_workspace_bytes(BZ_OP_VOTE_MEDIAN_HOST, r, f, d, 0, 0)) return BZ_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // slab of S coordinates: r*f input rows and one output row, each padded to a multiple of 64
    const size_t rows = static_cast<size_t>(r) * f + 1;
    int64_t S = static_cast<int64_t>(workspace_bytes / (rows * sizeof(float)));
    S = S / 64 * 64;
    if (S > (d + 63) / 64 * 64) S = (d + 63) / 64 * 64;
    float* slab = static_cast<float*>(workspace);
    float* out_dev = slab + static_cast<size_t>(r) * f * S;
    for (int64_t j0 = 0; j0 < d; j0 += S) {
        const int64_t n = (d - j0 < S) ? d - j0 : S;
        cudaError_t e = cudaMemcpy2DAsync(slab, S * sizeof(float), replicas_host + j0, d * sizeof(float),
                                          n * sizeof(float), static_cast<size_t>(r) * f, cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) return cuda_failed(e);
        st = vote_median_on_device(slab, r, f, n, S, static_cast<int64_t>(f) * S, out_dev, kNoUpdate, s);
        if (st != BZ_OK) return st;
        e = cudaMemcpyAsync(out_host + j0, out_dev, n * sizeof(float), cudaMemcpyDeviceToHost, s);
        if (e != cudaSuccess) return cuda_failed(e);
    }
    cudaError_t e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_failed(e);
    return BZ_OK;
}

namespace bz {
namespace {

__global__ void __launch_bounds__(256) model_update_kernel(const float* __restrict__ g, int64_t d, const ModelUpdate upd) {
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; j < d; j += stride)
        apply_update(upd, j, g[j]);
}

}  // namespace
}  // namespace bz

extern "C" int bz_vote_median_update(const float* replicas, int r, int f, int64_t d, int64_t ld_file,
                                     int64_t ld_replica, float* w, float* velocity, float eta, float mu, float* out,
                                     void* stream) {
    int st = validate_replicas(replicas, r, f, d, ld_file, ld_replica);
    if (st != BZ_OK) return st;
    if (w == nullptr && d > 0) return BZ_ERR_INVALID_ARG;
    if (d == 0) return BZ_OK;
    const ModelUpdate upd = {w, velocity, eta, mu};
    return vote_median_on_device(replicas, r, f, d, ld_file, ld_replica, out, upd, static_cast<cudaStream_t>(stream));
}

extern "C" int bz_model_update(const float* g, int64_t d, float* w, float* velocity, float eta, float mu, void* stream) {
    if (d < 0 || ((g == nullptr || w == nullptr) && d > 0)) return BZ_ERR_INVALID_ARG;
    if (d == 0) return BZ_OK;
    const ModelUpdate upd = {w, velocity, eta, mu};
    model_update_kernel<<<grid_for(d, 256, 8), 256, 0, static_cast<cudaStream_t>(stream)>>>(g, d, upd);
    note_launch();
    return check_launch();
}

extern "C" int bz_vote_median_rows(const float* const* rows, int r, int f, int64_t d, float* out, void* stream) {
    if (d < 0 || r < 1 || f < 1 || (r % 2) == 0 || rows == nullptr) return BZ_ERR_INVALID_ARG;
    if (r > BZ_MAX_R || f > BZ_MAX_F) return BZ_ERR_UNSUPPORTED;
    if (out == nullptr && d > 0) return BZ_ERR_INVALID_ARG;
    if (d == 0) return BZ_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int st = 1;
    switch (r) {
        case 1: st = vm_rows_dispatch_f<1>(rows, f, d, out, s); break;
        case 3: st = vm_rows_dispatch_f<3>(rows, f, d, out, s); break;
        case 5: st = vm_rows_dispatch_f<5>(rows, f, d, out, s); break;
        case 7: st = vm_rows_dispatch_f<7>(rows, f, d, out, s); break;
        default: break;
    }
    if (st != 1) return st;
    generic_rows_kernel<<<grid_for(d, 128, 8), 128, 0, s>>>(rows, r, f, d, nullptr, 0, out, 1);
    note_launch();
    return check_launch();
}

extern "C" int bz_vote_rows(const float* const* rows, int r, int f, int64_t d, float* voted, int64_t ld_voted, void* stream) {
    if (d < 0 || r < 1 || f < 1 || (r % 2) == 0 || rows == nullptr) return BZ_ERR_INVALID_ARG;
    if (r > BZ_MAX_R || f > BZ_MAX_F) return BZ_ERR_UNSUPPORTED;
    if ((voted == nullptr && d > 0) || ld_voted < d) return BZ_ERR_INVALID_ARG;
    if (d == 0) return BZ_OK;
    generic_rows_kernel<<<grid_for(d, 128, 8), 128, 0, static_cast<cudaStream_t>(stream)>>>(
        rows, r, f, d, reinterpret_cast<uint32_t*>(voted), ld_voted, nullptr, 0);
    note_launch();
    return check_launch();
}
