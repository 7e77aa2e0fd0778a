// Eq. (3) as the paper states it (Sec. 2, "Training Protocol"): per file, the WHOLE gradient that
// most of its r copies agree on, exact match on bit patterns; among equally frequent gradients the
// one whose first copy has the lowest index.  (bz_vote applies the same rule coordinate by
// coordinate; the two agree whenever a majority of a file's copies is identical.)
//
// Three kernels: (1) one streaming pass over the replicas that ORs, per file, a bit for every pair
// of copies that differ anywhere - and, on 16-byte aligned data, writes copy 0 to `voted` while it
// has it in registers; (2) a tiny kernel that turns the pair bits into the winner's index; (3) a
// gather of the winning copies into `voted`, which skips the files that copy 0 has won.  Bytes per
// coordinate: 4rf read and 4f written, then 8 more for every file whose first copy lost: bound by HBM.
#include "bz_common.cuh"

namespace bz {

namespace {

constexpr int kMaxPairs = BZ_MAX_R * (BZ_MAX_R - 1) / 2;   // 105: two 64-bit words per file
constexpr int kMaskWords = 2;

// When do two copies of a coordinate agree?  Exactly (bit patterns), or - for clusters whose honest
// members may differ by rounding (Sec. 2 suggests grouping such copies into clusters, without a rule) -
// within |a - b| <= abs_tol + rel_tol * max(|a|, |b|), evaluated in binary32 with one fused
// multiply-add; identical bit patterns always agree (so equal NaNs and infinities do).
struct Agreement {
    float abs_tol, rel_tol;
    int exact;
};
__device__ __forceinline__ bool differ1(uint32_t a, uint32_t b, const Agreement& g) {
    if (a == b) return false;
    if (g.exact) return true;
    const float x = __uint_as_float(a), y = __uint_as_float(b);
    const float gap = fabsf(__fsub_rn(x, y));
    const float bound = __fmaf_rn(g.rel_tol, fmaxf(fabsf(x), fabsf(y)), g.abs_tol);
    return !(gap <= bound);   // a NaN on either side differs
}
__device__ __forceinline__ bool differ(const uint4& a, const uint4& b, const Agreement& g) {
    if (g.exact) return ((a.x ^ b.x) | (a.y ^ b.y) | (a.z ^ b.z) | (a.w ^ b.w)) != 0;
    return differ1(a.x, b.x, g) || differ1(a.y, b.y, g) || differ1(a.z, b.z, g) || differ1(a.w, b.w, g);
}
__device__ __forceinline__ bool differ(uint32_t a, uint32_t b, const Agreement& g) { return differ1(a, b, g); }
// the same test out of line: the streaming kernel calls it only for pairs that its quick test could not pass
__device__ __noinline__ bool differ_exactly(const uint4 a, const uint4 b, const Agreement g) { return differ(a, b, g); }
__device__ __noinline__ bool differ_exactly(const uint32_t a, const uint32_t b, const Agreement g) { return differ1(a, b, g); }

// the smaller of a and b; a NaN in either comes through
__device__ __forceinline__ float min_nan(float a, float b) {
    float m;
    asm("min.NaN.f32 %0, %1, %2;" : "=f"(m) : "f"(a), "f"(b));
    return m;
}
__device__ __forceinline__ void unpack(const uint4& v, float (&o)[4]) {
    o[0] = __uint_as_float(v.x);
    o[1] = __uint_as_float(v.y);
    o[2] = __uint_as_float(v.z);
    o[3] = __uint_as_float(v.w);
}
__device__ __forceinline__ void unpack(uint32_t v, float (&o)[1]) { o[0] = __uint_as_float(v); }

// pair (k, k2), k < k2, -> bit index, row-major over the strict upper triangle
__host__ __device__ __forceinline__ int pair_index(int r, int k, int k2) { return k * r - k * (k + 1) / 2 + (k2 - k - 1); }

// grid = (chunks, f).  V = uint4: n counts groups of 4 coordinates and leading dimensions are in groups.
template <int R, typename V, bool EXACT>
__global__ void __launch_bounds__(256) copies_differ_kernel(const V* __restrict__ rep, int64_t n, int64_t ld_file, int64_t ld_rep,
                                                            unsigned long long* __restrict__ mask, const Agreement agree,
                                                            V* __restrict__ voted, int64_t ld_voted) {
    const int file = blockIdx.y;
    const V* base = rep + file * ld_file;
    V* first = voted != nullptr ? voted + file * ld_voted : nullptr;  // copy 0 goes here: right unless it loses
    uint32_t bits = 0;  // R <= 7: 21 pairs
#pragma unroll 2
    for (int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; j < n; j += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        V c[R];
#pragma unroll
        for (int k = 0; k < R; ++k) c[k] = ld_stream(base + k * ld_rep + j);
        if (first != nullptr) st_stream(first + j, c[0]);
        int p = 0;
        if constexpr (EXACT) {
#pragma unroll
            for (int k = 0; k < R; ++k)
#pragma unroll
                for (int k2 = k + 1; k2 < R; ++k2, ++p) bits |= differ(c[k], c[k2], agree) ? (1u << p) : 0u;
        } else {
            // The bound abs_tol + rel_tol*max(|a|, |b|) is the larger of the two copies' own bounds (the
            // multiply-add is monotone in |a|), so each copy's bound is formed once.  A pair passes at once
            // if its smallest margin bound - |a - b| is >= 0; anything else (a real difference, or NaN /
            // infinities, whose margin is NaN) goes to the exact test.  A pair this thread has already
            // seen differ is not looked at again.
            constexpr int VE = sizeof(V) / 4;
            float x[R][VE], bound[R][VE];
#pragma unroll
            for (int k = 0; k < R; ++k) {
                unpack(c[k], x[k]);
#pragma unroll
                for (int e = 0; e < VE; ++e) {
                    bound[k][e] = __fmaf_rn(agree.rel_tol, fabsf(x[k][e]), agree.abs_tol);
                }
            }
#pragma unroll
            for (int k = 0; k < R; ++k)
#pragma unroll
                for (int k2 = k + 1; k2 < R; ++k2, ++p) {
                    if (((bits >> p) & 1u) == 0) {
                        float least = __int_as_float(0x7f800000);
#pragma unroll
                        for (int e = 0; e < VE; ++e)
                            least = min_nan(least, __fsub_rn(fmaxf(bound[k][e], bound[k2][e]), fabsf(__fsub_rn(x[k][e], x[k2][e]))));
                        if (!(least >= 0.f) && differ_exactly(c[k], c[k2], agree)) bits |= 1u << p;
                    }
                }
        }
    }
    bits = __reduce_or_sync(0xffffffffu, bits);
    if ((threadIdx.x & 31) == 0 && bits != 0) atomicOr(&mask[file * kMaskWords], static_cast<unsigned long long>(bits));
}

// any odd r <= BZ_MAX_R, any alignment
__global__ void __launch_bounds__(256) copies_differ_generic_kernel(const uint32_t* __restrict__ rep, int r, int64_t d, int64_t ld_file,
                                                                    int64_t ld_rep, unsigned long long* __restrict__ mask,
                                                                    const Agreement agree) {
    const int file = blockIdx.y;
    const uint32_t* base = rep + file * ld_file;
    unsigned long long lo = 0, hi = 0;
    for (int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; j < d; j += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        uint32_t c[BZ_MAX_R];
        for (int k = 0; k < r; ++k) c[k] = base[k * ld_rep + j];
        int p = 0;
        for (int k = 0; k < r; ++k)
            for (int k2 = k + 1; k2 < r; ++k2, ++p)
                if (differ1(c[k], c[k2], agree)) {
                    if (p < 64) lo |= 1ull << p;
                    else hi |= 1ull << (p - 64);
                }
    }
    if (lo) atomicOr(&mask[file * kMaskWords], lo);
    if (hi) atomicOr(&mask[file * kMaskWords + 1], hi);
}

// thread i: winner of file i from its pair bits
__global__ void __launch_bounds__(BZ_MAX_F) winner_kernel(const unsigned long long* __restrict__ mask, int r, int f,
                                                          int32_t* __restrict__ winner) {
    const int i = threadIdx.x;
    if (i >= f) return;
    const unsigned long long lo = mask[i * kMaskWords], hi = mask[i * kMaskWords + 1];
    auto same = [&](int k, int k2) {
        if (k == k2) return true;
        const int p = k < k2 ? pair_index(r, k, k2) : pair_index(r, k2, k);
        return ((p < 64 ? lo >> p : hi >> (p - 64)) & 1ull) == 0;
    };
    int best = 0, best_count = 0;
    for (int k = 0; k < r; ++k) {
        int count = 0;
        for (int k2 = 0; k2 < r; ++k2) count += same(k, k2) ? 1 : 0;
        if (count > best_count) {
            best_count = count;
            best = k;
        }
    }
    winner[i] = best;
}

template <typename V>
__global__ void __launch_bounds__(256) gather_winners_kernel(const V* __restrict__ rep, int64_t n, int64_t ld_file, int64_t ld_rep,
                                                             const int32_t* __restrict__ winner, V* __restrict__ voted, int64_t ld_voted,
                                                             int have_copy0) {
    const int file = blockIdx.y;
    if (have_copy0 && winner[file] == 0) return;  // the first pass has written this row
    const V* src = rep + winner[file] * ld_rep + file * ld_file;
    V* dst = voted + file * ld_voted;
    // few files may be left to copy, so every thread keeps four loads in flight
    const int64_t step = static_cast<int64_t>(gridDim.x) * blockDim.x;
    int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    for (; j + 3 * step < n; j += 4 * step) {
        const V x0 = ld_stream(src + j), x1 = ld_stream(src + j + step), x2 = ld_stream(src + j + 2 * step), x3 = ld_stream(src + j + 3 * step);
        st_stream(dst + j, x0);
        st_stream(dst + j + step, x1);
        st_stream(dst + j + 2 * step, x2);
        st_stream(dst + j + 3 * step, x3);
    }
    for (; j < n; j += step) st_stream(dst + j, ld_stream(src + j));
}

int chunks_for(int64_t n, int f) {
    // enough CTAs to fill the SMs a few times over, never more than the work
    int64_t per_file = (static_cast<int64_t>(kNumSMs) * 8 + f - 1) / f;
    const int64_t most = (n + 255) / 256;
    if (per_file > most) per_file = most;
    if (per_file < 1) per_file = 1;
    return static_cast<int>(per_file);
}

template <int R>
int launch_differ_vec(const float* rep, int f, int64_t d, int64_t ld_file, int64_t ld_rep, unsigned long long* mask,
                      const Agreement& agree, float* voted, int64_t ld_voted, cudaStream_t s) {
    const int64_t n = d / 4;
    const dim3 grid(chunks_for(n, f), f);
    if (agree.exact)
        copies_differ_kernel<R, uint4, true><<<grid, 256, 0, s>>>(reinterpret_cast<const uint4*>(rep), n, ld_file / 4, ld_rep / 4, mask, agree,
                                                                  reinterpret_cast<uint4*>(voted), ld_voted / 4);
    else
        copies_differ_kernel<R, uint4, false><<<grid, 256, 0, s>>>(reinterpret_cast<const uint4*>(rep), n, ld_file / 4, ld_rep / 4, mask, agree,
                                                                   reinterpret_cast<uint4*>(voted), ld_voted / 4);
    note_launch();
    return check_launch();
}

}  // namespace

size_t vote_vectorwise_workspace(int f) { return round_up(static_cast<size_t>(f) * (kMaskWords * 8 + 4), 256); }

}  // namespace bz

using namespace bz;

static int vote_whole_vectors(const float* replicas, int r, int f, int64_t d, int64_t ld_file, int64_t ld_replica, float* voted,
                              int64_t ld_voted, int32_t* winner, void* workspace, size_t workspace_bytes, const Agreement& agree,
                              void* stream) {
    // the argument rules of bz_vote
    if (d < 0 || r < 1 || f < 1 || (r % 2) == 0) return BZ_ERR_INVALID_ARG;
    if (replicas == nullptr && d > 0) return BZ_ERR_INVALID_ARG;
    if (r > BZ_MAX_R || f > BZ_MAX_F) return BZ_ERR_UNSUPPORTED;
    if (ld_file < d || (r > 1 && ld_replica < d)) return BZ_ERR_INVALID_ARG;
    int st = BZ_OK;
    if (voted == nullptr && winner == nullptr) return BZ_ERR_INVALID_ARG;
    if (voted != nullptr && ld_voted < d) return BZ_ERR_INVALID_ARG;
    if (workspace == nullptr || !aligned256(workspace) || workspace_bytes < vote_vectorwise_workspace(f)) return BZ_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned long long* mask = static_cast<unsigned long long*>(workspace);
    int32_t* win = winner != nullptr ? winner : reinterpret_cast<int32_t*>(mask + static_cast<size_t>(f) * kMaskWords);
    cudaError_t e = cudaMemsetAsync(mask, 0, static_cast<size_t>(f) * kMaskWords * 8, s);  // every call starts from "all copies agree"
    if (e != cudaSuccess) return cuda_failed(e);
    int have_copy0 = 0;
    if (d > 0 && r > 1) {
        const bool vec = aligned16(replicas) && (ld_file % 4 == 0) && (ld_replica % 4 == 0) && (d % 4 == 0) && (r == 3 || r == 5 || r == 7);
        if (vec) {
            float* first = (voted != nullptr && aligned16(voted) && ld_voted % 4 == 0) ? voted : nullptr;
            have_copy0 = first != nullptr;
            st = r == 3 ? launch_differ_vec<3>(replicas, f, d, ld_file, ld_replica, mask, agree, first, ld_voted, s)
                        : (r == 5 ? launch_differ_vec<5>(replicas, f, d, ld_file, ld_replica, mask, agree, first, ld_voted, s)
                                  : launch_differ_vec<7>(replicas, f, d, ld_file, ld_replica, mask, agree, first, ld_voted, s));
        } else {
            const dim3 grid(chunks_for(d, f), f);
            copies_differ_generic_kernel<<<grid, 256, 0, s>>>(reinterpret_cast<const uint32_t*>(replicas), r, d, ld_file, ld_replica, mask, agree);
            note_launch();
            st = check_launch();
        }
        if (st != BZ_OK) return st;
    }
    winner_kernel<<<1, BZ_MAX_F, 0, s>>>(mask, r, f, win);
    note_launch();
    st = check_launch();
    if (st != BZ_OK || voted == nullptr || d == 0) return st;
    const bool vec = aligned16(replicas) && aligned16(voted) && (ld_file % 4 == 0) && (ld_voted % 4 == 0) && (d % 4 == 0) &&
                     (r == 1 || ld_replica % 4 == 0);
    if (vec) {
        const dim3 grid(chunks_for(d / 4, f), f);
        gather_winners_kernel<uint4><<<grid, 256, 0, s>>>(reinterpret_cast<const uint4*>(replicas), d / 4, ld_file / 4, ld_replica / 4, win,
                                                          reinterpret_cast<uint4*>(voted), ld_voted / 4, have_copy0);
    } else {
        const dim3 grid(chunks_for(d, f), f);
        gather_winners_kernel<uint32_t><<<grid, 256, 0, s>>>(reinterpret_cast<const uint32_t*>(replicas), d, ld_file, ld_replica, win,
                                                             reinterpret_cast<uint32_t*>(voted), ld_voted, have_copy0);
    }
    note_launch();
    return check_launch();
}

extern "C" int bz_vote_vectorwise(const float* replicas, int r, int f, int64_t d, int64_t ld_file, int64_t ld_replica, float* voted,
                                  int64_t ld_voted, int32_t* winner, void* workspace, size_t workspace_bytes, void* stream) {
    const Agreement exact{0.f, 0.f, 1};
    return vote_whole_vectors(replicas, r, f, d, ld_file, ld_replica, voted, ld_voted, winner, workspace, workspace_bytes, exact, stream);
}

extern "C" int bz_vote_clusters(const float* replicas, int r, int f, int64_t d, int64_t ld_file, int64_t ld_replica, float abs_tol,
                                float rel_tol, float* voted, int64_t ld_voted, int32_t* winner, void* workspace,
                                size_t workspace_bytes, void* stream) {
    if (!(abs_tol >= 0.f) || !(rel_tol >= 0.f)) return BZ_ERR_INVALID_ARG;  // negative or NaN tolerances
    const Agreement within{abs_tol, rel_tol, 0};
    return vote_whole_vectors(replicas, r, f, d, ld_file, ld_replica, voted, ld_voted, winner, workspace, workspace_bytes, within, stream);
}
