// Exhaustive worst-case search (Sec. 5.3.2, Sec. 6.1): over all q-subsets S of the K workers, the
// largest number of files whose majority (r' = (r+1)/2 of r holders) lies inside S.
//
// Every worker is a 64-bit mask of the files it holds.  The number of holders of each file inside
// S is kept bit-sliced in three 64-bit planes (counts 0..7, enough for r <= 7): adding a worker is
// a ripple-carry add of its mask, the threshold ">= r'" is a Boolean function of the planes and the
// answer is one popcount.  Threads take fixed-size runs of consecutive lexicographic ranks, unrank
// the first subset of a run with the combinatorial number system and then walk successors,
// keeping the plane state of every prefix so that a successor only redoes the changed suffix.
#include "bz_common.cuh"

namespace bz {

namespace {

constexpr int kMaxK = 64;
constexpr int kMaxQ = 64;
constexpr int kWcBlock = 128;
constexpr uint64_t kRun = 2048;  // subsets per run

struct Planes {
    uint64_t c0, c1, c2;
};

__device__ __forceinline__ Planes add_mask(const Planes& s, uint64_t m) {
    Planes o;
    o.c0 = s.c0 ^ m;
    const uint64_t k0 = s.c0 & m;
    o.c1 = s.c1 ^ k0;
    const uint64_t k1 = s.c1 & k0;
    o.c2 = s.c2 ^ k1;
    return o;
}

// files with at least rp holders (rp in 1..4)
__device__ __forceinline__ int count_at_least(const Planes& s, int rp) {
    uint64_t hit;
    if (rp == 1)
        hit = s.c0 | s.c1 | s.c2;
    else if (rp == 2)
        hit = s.c1 | s.c2;
    else if (rp == 3)
        hit = s.c2 | (s.c1 & s.c0);
    else
        hit = s.c2;
    return __popcll(hit);
}

struct WcParams {
    uint64_t mask[kMaxK];
    uint64_t total;  // C(K, q)
    int K, q, rp;
};

struct WcResult {
    // a larger (count, members) pair is a better answer: count first, then the lexicographically
    // earlier subset (worker u is bit 63-u of `members`, so an earlier subset is a larger integer)
    uint32_t count;
    uint32_t pad;
    uint64_t members;
};

__device__ __forceinline__ bool better(uint32_t c1, uint64_t m1, uint32_t c2, uint64_t m2) {
    return c1 > c2 || (c1 == c2 && m1 > m2);
}

// binom[n][k] for n, k <= 64 (saturating), filled by the host into constant memory
__constant__ uint64_t c_binom[kMaxK + 1][kMaxK + 1];

__global__ void __launch_bounds__(kWcBlock)
    worst_case_kernel(const __grid_constant__ WcParams prm, WcResult* __restrict__ results) {
    __shared__ uint64_t s_mask[kMaxK];
    __shared__ uint32_t s_cnt[kWcBlock];
    __shared__ uint64_t s_mem[kWcBlock];
    for (int u = threadIdx.x; u < prm.K; u += blockDim.x) s_mask[u] = prm.mask[u];
    __syncthreads();

    const int K = prm.K, q = prm.q, rp = prm.rp;
    uint32_t best_cnt = 0;
    uint64_t best_mem = 0;
    bool have = false;

    int comb[kMaxQ];
    Planes prefix[kMaxQ];  // prefix[i] = planes of comb[0..i-1]

    const uint64_t n_runs = (prm.total + kRun - 1) / kRun;
    const uint64_t first_run = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const uint64_t run_stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    for (uint64_t run = first_run; run < n_runs; run += run_stride) {
        const uint64_t rank = run * kRun;
        uint64_t left = prm.total - rank < kRun ? prm.total - rank : kRun;
        // unrank: the rank-th q-subset in lexicographic order
        {
            int x = 0;
            uint64_t rest = rank;
            for (int i = 0; i < q; ++i) {
                // subsets whose element i is x (earlier elements fixed): C(K-1-x, q-1-i)
                while (true) {
                    const uint64_t cnt = c_binom[K - 1 - x][q - 1 - i];
                    if (rest < cnt) break;
                    rest -= cnt;
                    ++x;
                }
                comb[i] = x++;
            }
        }
        prefix[0] = Planes{0, 0, 0};
        for (int i = 0; i + 1 < q; ++i) prefix[i + 1] = add_mask(prefix[i], s_mask[comb[i]]);

        while (true) {
            // last position: sweep its remaining values with the prefix state fixed
            const Planes base = prefix[q - 1];
            for (int x = comb[q - 1]; x < K && left > 0; ++x, --left) {
                const uint32_t cnt = static_cast<uint32_t>(count_at_least(add_mask(base, s_mask[x]), rp));
                // a thread meets subsets in lexicographic order: only a larger count replaces
                if (!have || cnt > best_cnt) {
                    uint64_t mem = 1ull << (63 - x);
                    for (int i = 0; i + 1 < q; ++i) mem |= 1ull << (63 - comb[i]);
                    best_cnt = cnt;
                    best_mem = mem;
                    have = true;
                }
            }
            if (left == 0) break;
            // successor of the prefix comb[0..q-2]
            int i = q - 2;
            while (i >= 0 && comb[i] == K - q + i) --i;
            if (i < 0) break;  // the last subset was reached; cannot happen while left > 0
            ++comb[i];
            for (int t = i + 1; t < q; ++t) comb[t] = comb[t - 1] + 1;
            for (int t = i; t + 1 < q; ++t) prefix[t + 1] = add_mask(prefix[t], s_mask[comb[t]]);
        }
    }

    // threads interleave their runs: reduce with the full (count, members) order
    s_cnt[threadIdx.x] = have ? best_cnt : 0;
    s_mem[threadIdx.x] = have ? best_mem : 0;
    __syncthreads();
    for (int off = kWcBlock / 2; off > 0; off >>= 1) {
        if (threadIdx.x < off &&
            better(s_cnt[threadIdx.x + off], s_mem[threadIdx.x + off], s_cnt[threadIdx.x], s_mem[threadIdx.x])) {
            s_cnt[threadIdx.x] = s_cnt[threadIdx.x + off];
            s_mem[threadIdx.x] = s_mem[threadIdx.x + off];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        results[blockIdx.x].count = s_cnt[0];
        results[blockIdx.x].pad = 0;
        results[blockIdx.x].members = s_mem[0];
    }
}

constexpr int kWcMaxBlocks = kNumSMs * 8;

uint64_t h_binom[kMaxK + 1][kMaxK + 1];
bool binom_ready = false;

int upload_binom() {
    if (!binom_ready) {
        for (int n = 0; n <= kMaxK; ++n)
            for (int k = 0; k <= kMaxK; ++k) {
                if (k == 0)
                    h_binom[n][k] = 1;
                else if (n == 0)
                    h_binom[n][k] = 0;
                else {
                    const uint64_t a = h_binom[n - 1][k - 1], b = h_binom[n - 1][k];
                    h_binom[n][k] = (a > UINT64_MAX - b) ? UINT64_MAX : a + b;
                }
            }
        binom_ready = true;
    }
    const cudaError_t e = cudaMemcpyToSymbol(c_binom, h_binom, sizeof(h_binom));
    if (e != cudaSuccess) return cuda_failed(e);
    return BZ_OK;
}

}  // namespace

size_t worst_case_workspace_bytes() { return round_up(sizeof(WcResult) * kWcMaxBlocks, 256); }

}  // namespace bz

using namespace bz;

extern "C" int bz_worst_case(const uint64_t* worker_mask, int K, int f, int r, int q, uint64_t max_subsets,
                             int32_t* c_max, int32_t* argmax, uint64_t* n_subsets, void* workspace,
                             size_t workspace_bytes, void* stream) {
    if (worker_mask == nullptr || c_max == nullptr) return BZ_ERR_INVALID_ARG;
    if (K < 1 || f < 1 || r < 1 || (r % 2) == 0 || q < 0 || q > K) return BZ_ERR_INVALID_ARG;
    if (K > kMaxK || f > 64 || r > 7) return BZ_ERR_UNSUPPORTED;
    if (f < 64)
        for (int u = 0; u < K; ++u)
            if (worker_mask[u] >> f) return BZ_ERR_INVALID_ARG;
    if (workspace == nullptr || !aligned256(workspace) || workspace_bytes < worst_case_workspace_bytes())
        return BZ_ERR_WORKSPACE;
    int st = upload_binom();
    if (st != BZ_OK) return st;
    const uint64_t total = h_binom[K][q];
    if (total == UINT64_MAX) return BZ_ERR_BUDGET;
    if (max_subsets != 0 && total > max_subsets) return BZ_ERR_BUDGET;
    if (n_subsets) *n_subsets = total;
    if (q == 0) {
        *c_max = 0;
        return BZ_OK;
    }
    WcParams prm;
    for (int u = 0; u < kMaxK; ++u) prm.mask[u] = u < K ? worker_mask[u] : 0;
    prm.total = total;
    prm.K = K;
    prm.q = q;
    prm.rp = (r + 1) / 2;
    const uint64_t n_runs = (total + kRun - 1) / kRun;
    uint64_t blocks = (n_runs + kWcBlock - 1) / kWcBlock;
    if (blocks > static_cast<uint64_t>(kWcMaxBlocks)) blocks = kWcMaxBlocks;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    WcResult* dev = static_cast<WcResult*>(workspace);
    worst_case_kernel<<<static_cast<int>(blocks), kWcBlock, 0, s>>>(prm, dev);
    note_launch();
    st = check_launch();
    if (st != BZ_OK) return st;
    static thread_local WcResult host[kWcMaxBlocks];
    cudaError_t e = cudaMemcpyAsync(host, dev, sizeof(WcResult) * blocks, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_failed(e);
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_failed(e);
    uint32_t best_cnt = host[0].count;
    uint64_t best_mem = host[0].members;
    for (uint64_t b = 1; b < blocks; ++b)
        if (host[b].count > best_cnt || (host[b].count == best_cnt && host[b].members > best_mem)) {
            best_cnt = host[b].count;
            best_mem = host[b].members;
        }
    *c_max = static_cast<int32_t>(best_cnt);
    if (argmax) {
        int t = 0;
        for (int u = 0; u < K && t < q; ++u)
            if (best_mem & (1ull << (63 - u))) argmax[t++] = u;
    }
    return BZ_OK;
}
