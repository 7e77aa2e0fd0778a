// Exhaustive worst-case search (Sec. 5.3.2, Sec. 6.1): over all q-subsets S of the K workers, the
// largest number of files whose majority (r' = (r+1)/2 of r holders) lies inside S.
//
// Every worker is a 64-bit mask of the files it holds.  The number of holders of each file inside
// S is kept bit-sliced in three 64-bit planes (counts 0..7, enough for r <= 7): adding a worker is
// a ripple-carry add of its mask, the threshold ">= r'" is a Boolean function of the planes and the
// answer is one popcount.
//
// Enumeration: a subset is a prefix of p = q - T workers followed by a tail of T <= 5 workers.  The
// tail is T nested loops with all state in registers; in the innermost one a subset costs a
// load, an AND and a popcount, and the loop above it updates count and mask without a bit-sliced add.  Prefixes are grouped by their largest worker l: inside a group every prefix has the same
// tail range (l, K), so the threads of a warp run the nested loops with identical trip counts.  A
// group's prefixes are l plus the (p-1)-subsets of {0..l-1}; threads take chunks of consecutive
// ones, unrank the first with the combinatorial number system and walk lexicographic successors,
// keeping the plane state of every prefix length so that a successor redoes only the changed suffix.
// The answer is the largest (count, membership mask with worker u at bit 63-u): the larger mask is
// the lexicographically earlier subset, so ties resolve to the first maximiser whatever the order
// of enumeration.
#include "worst_case_common.cuh"

namespace bz {

namespace {

constexpr int kMaxK = 64;
constexpr int kMaxQ = 64;
constexpr int kMaxTail = 5;
constexpr uint64_t kSubsetsPerChunk = 16384;  // target work per chunk

// tail workers chosen by the enclosing loops (outermost first); only read when a candidate is offered
struct TailIds {
    int w[4];
};

__device__ __forceinline__ uint64_t member_bits(uint64_t prefix_mem, const TailIds& ids, int n_ids, int x) {
    uint64_t mem = prefix_mem | (1ull << (63 - x));
    for (int i = 0; i < n_ids; ++i) mem |= 1ull << (63 - ids.w[i]);
    return mem;
}

// innermost loop: adding worker x distorts exactly the files that were one holder short (`tip`), so the
// count under each x is the count of the enclosing subset (`base`) plus one popcount
template <int DEPTH>
__device__ __forceinline__ void leaf_loop(const uint64_t* __restrict__ s_mask, int base, uint64_t tip, int x_lo, int x_hi,
                                          uint64_t prefix_mem, const TailIds& ids, Best& best) {
    for (int x = x_lo; x < x_hi; ++x) {
        const int cnt = base + __popcll(s_mask[x] & tip);
        if (cnt >= best.cnt) offer(best, cnt, member_bits(prefix_mem, ids, DEPTH, x));
    }
}

// The loop above the innermost one needs no bit-sliced add either: with worker y added, the count grows by the
// one-short files y holds, and the new one-short files are the old ones y does not hold plus the two-short ones
// it does.
template <int DEPTH>
__device__ __forceinline__ void pair_loops(const uint64_t* __restrict__ s_mask, int base, uint64_t tip1, uint64_t tip2, int y_lo,
                                           int y_hi, int K, uint64_t prefix_mem, TailIds& ids, Best& best) {
    for (int y = y_lo; y < y_hi; ++y) {
        ids.w[DEPTH] = y;
        const uint64_t m = s_mask[y];
        leaf_loop<DEPTH + 1>(s_mask, base + __popcll(tip1 & m), (tip1 & ~m) | (tip2 & m), y + 1, K, prefix_mem, ids, best);
    }
}

// LEVEL nested loops over the tail workers start <= w_1 < ... < w_LEVEL < K
template <int RP, int LEVEL, int DEPTH>
__device__ __forceinline__ void tail_loops(const uint64_t* __restrict__ s_mask, const Planes& s, int start, int K,
                                           uint64_t prefix_mem, TailIds& ids, Best& best) {
    if constexpr (LEVEL == 1) {
        leaf_loop<DEPTH>(s_mask, count_at_least<RP>(s), one_short<RP>(s), start, K, prefix_mem, ids, best);
    } else if constexpr (LEVEL == 2) {
        pair_loops<DEPTH>(s_mask, count_at_least<RP>(s), one_short<RP>(s), two_short<RP>(s), start, K - 1, K, prefix_mem, ids, best);
    } else {
        for (int y = start; y <= K - LEVEL; ++y) {
            ids.w[DEPTH] = y;
            tail_loops<RP, LEVEL - 1, DEPTH + 1>(s_mask, add_mask(s, s_mask[y]), y + 1, K, prefix_mem, ids, best);
        }
    }
}

// the outermost tail loop restricted to [y_lo, y_hi)
template <int RP, int LEVEL>
__device__ __forceinline__ void tail_top(const uint64_t* __restrict__ s_mask, const Planes& s, int y_lo, int y_hi, int K,
                                         uint64_t mem, Best& best) {
    TailIds ids;
    if constexpr (LEVEL == 1) {
        leaf_loop<0>(s_mask, count_at_least<RP>(s), one_short<RP>(s), y_lo, y_hi, mem, ids, best);
    } else if constexpr (LEVEL == 2) {
        pair_loops<0>(s_mask, count_at_least<RP>(s), one_short<RP>(s), two_short<RP>(s), y_lo, y_hi, K, mem, ids, best);
    } else {
        for (int y = y_lo; y < y_hi; ++y) {
            ids.w[0] = y;
            tail_loops<RP, LEVEL - 1, 1>(s_mask, add_mask(s, s_mask[y]), y + 1, K, mem, ids, best);
        }
    }
}

// A group (all prefixes with the same largest worker) is cut into chunks along two axes: runs of
// chunk_len consecutive prefixes, and - where one prefix alone has too many tails - pieces of y_width
// values of the first tail worker.  Chunk index = piece * prefix_chunks + run, so neighbouring
// threads hold neighbouring prefix runs of the same piece and loop in step.
struct WcParams {
    uint64_t mask[kMaxK];
    uint64_t chunk_begin[kMaxK + 1];   // first chunk of each group; chunk_begin[n_groups] = number of chunks
    uint64_t prefix_chunks[kMaxK];     // runs of prefixes in each group
    uint32_t chunk_len[kMaxK];         // prefixes per run
    uint32_t y_width[kMaxK];           // first-tail-worker values per piece
    int K, q, p, n_groups, first_l;   // group g holds the prefixes whose largest worker is first_l + g
    uint32_t part, parts;             // this launch takes the chunks whose index is part modulo parts
};

// binom[n][k] for n, k <= 64 (saturating), filled by the host into constant memory
__constant__ uint64_t c_binom[kMaxK + 1][kMaxK + 1];

template <int RP, int T>
__global__ void __launch_bounds__(kWcBlock, 12)
    worst_case_kernel(const __grid_constant__ WcParams prm, WcResult* __restrict__ results) {
    __shared__ uint64_t s_mask[kMaxK];
    __shared__ uint64_t s_begin[kMaxK + 1];
    __shared__ int32_t s_cnt[kWcBlock];
    __shared__ uint64_t s_mem[kWcBlock];
    for (int u = threadIdx.x; u < prm.K; u += blockDim.x) s_mask[u] = prm.mask[u];
    for (int u = threadIdx.x; u <= prm.n_groups; u += blockDim.x) s_begin[u] = prm.chunk_begin[u];
    __syncthreads();

    const int K = prm.K, p = prm.p;
    Best best{-1, 0};
    int comb[kMaxQ];
    Planes state[kMaxQ + 1];  // state[i] = planes of comb[0..i-1]

    const uint64_t n_chunks = s_begin[prm.n_groups];
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    int g = 0;
    for (uint64_t unit = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x;; unit += stride) {
        const uint64_t chunk = prm.part + prm.parts * unit;
        if (chunk >= n_chunks) break;
        while (chunk >= s_begin[g + 1]) ++g;  // chunks only move forward
        const int l = prm.first_l + g;        // largest worker of the prefix (p >= 1), or -1 when p == 0
        const int m = p - 1;                  // free prefix elements, from {0..l-1}
        const uint64_t in_group = m > 0 ? c_binom[l][m] : 1;
        const uint64_t in_g = chunk - s_begin[g];
        const uint64_t piece = in_g / prm.prefix_chunks[g];
        const uint64_t rank = (in_g - piece * prm.prefix_chunks[g]) * prm.chunk_len[g];
        const int y_lo = l + 1 + static_cast<int>(piece) * static_cast<int>(prm.y_width[g]);
        const int y_end = K - T + 1;  // the first tail worker leaves room for the other T-1
        const int y_hi = y_lo + static_cast<int>(prm.y_width[g]) < y_end ? y_lo + static_cast<int>(prm.y_width[g]) : y_end;
        uint64_t left = in_group - rank < prm.chunk_len[g] ? in_group - rank : prm.chunk_len[g];
        // unrank: the rank-th m-subset of {0..l-1} in lexicographic order
        {
            int x = 0;
            uint64_t rest = rank;
            for (int i = 0; i < m; ++i) {
                while (true) {
                    const uint64_t cnt = c_binom[l - 1 - x][m - 1 - i];  // subsets whose element i is x
                    if (rest < cnt) break;
                    rest -= cnt;
                    ++x;
                }
                comb[i] = x++;
            }
        }
        if (p > 0) comb[p - 1] = l;
        state[0] = Planes{0, 0, 0};
        for (int i = 0; i < p; ++i) state[i + 1] = add_mask(state[i], s_mask[comb[i]]);

        while (true) {
            uint64_t mem = 0;
            for (int i = 0; i < p; ++i) mem |= 1ull << (63 - comb[i]);
            tail_top<RP, T>(s_mask, state[p], y_lo, y_hi, K, mem, best);
            if (--left == 0) break;
            // successor of the free elements inside {0..l-1}
            int i = m - 1;
            while (i >= 0 && comb[i] == l - m + i) --i;
            if (i < 0) break;  // the group's last prefix; cannot happen while left > 0
            ++comb[i];
            for (int t = i + 1; t < m; ++t) comb[t] = comb[t - 1] + 1;
            for (int t = i; t < p; ++t) state[t + 1] = add_mask(state[t], s_mask[comb[t]]);
        }
    }

    block_best(best, s_cnt, s_mem, results);
}


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

template <int RP>
void launch_tail(int tail, int grid, cudaStream_t s, const WcParams& prm, WcResult* dev) {
    switch (tail) {
        case 1: worst_case_kernel<RP, 1><<<grid, kWcBlock, 0, s>>>(prm, dev); break;
        case 2: worst_case_kernel<RP, 2><<<grid, kWcBlock, 0, s>>>(prm, dev); break;
        case 3: worst_case_kernel<RP, 3><<<grid, kWcBlock, 0, s>>>(prm, dev); break;
        case 4: worst_case_kernel<RP, 4><<<grid, kWcBlock, 0, s>>>(prm, dev); break;
        default: worst_case_kernel<RP, 5><<<grid, kWcBlock, 0, s>>>(prm, dev); break;
    }
}

}  // namespace

size_t worst_case_workspace_bytes() { return round_up(sizeof(WcResult) * kWcMaxBlocks, 256); }

}  // namespace bz

using namespace bz;

// The search over the chunks whose index is `part` modulo `parts` (the whole search: 0 of 1).  A share without
// a chunk reports c_max = -1.
static int worst_case_share(const uint64_t* worker_mask, int K, int f, int r, int q, int part, int parts, uint64_t max_subsets,
                            int32_t* c_max, int32_t* argmax, uint64_t* n_subsets, void* workspace, size_t workspace_bytes,
                            void* stream) {
    if (worker_mask == nullptr || c_max == nullptr) return BZ_ERR_INVALID_ARG;
    if (parts < 1 || part < 0 || part >= parts) return BZ_ERR_INVALID_ARG;
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
        *c_max = part == 0 ? 0 : -1;  // the one (empty) set belongs to the first share
        return BZ_OK;
    }
    WcParams prm;
    prm.part = static_cast<uint32_t>(part);
    prm.parts = static_cast<uint32_t>(parts);
    for (int u = 0; u < kMaxK; ++u) prm.mask[u] = u < K ? worker_mask[u] : 0;
    const int tail = q < kMaxTail ? q : kMaxTail;
    const int p = q - tail;
    prm.K = K;
    prm.q = q;
    prm.p = p;
    // chunk size: about kSubsetsPerChunk subsets, fewer when the whole search is small
    uint64_t per_chunk = total / (static_cast<uint64_t>(kWcMaxBlocks) * kWcBlock * 4);
    if (per_chunk > kSubsetsPerChunk) per_chunk = kSubsetsPerChunk;
    if (per_chunk < 512) per_chunk = 512;
    uint64_t n_chunks = 0;
    // group g: prefixes whose largest worker is l = first_l + g (p == 0: the empty prefix, l = -1)
    prm.first_l = p - 1;
    prm.n_groups = p == 0 ? 1 : (K - tail - 1) - (p - 1) + 1;
    for (int g = 0; g < prm.n_groups; ++g) {
        const int l = prm.first_l + g;
        const uint64_t prefixes = p == 0 ? 1 : h_binom[l][p - 1];
        const uint64_t tails = h_binom[K - 1 - l][tail];
        const int n_y = K - tail - l;  // values of the first tail worker
        uint64_t len = 1, width = static_cast<uint64_t>(n_y);
        if (tails <= per_chunk) {
            len = per_chunk / tails;
        } else {
            // tails under the first value of the first tail worker (the largest share)
            const uint64_t under_first = h_binom[K - 2 - l][tail - 1];
            width = per_chunk / under_first;
            if (width < 1) width = 1;
            if (width > static_cast<uint64_t>(n_y)) width = static_cast<uint64_t>(n_y);
        }
        if (len > 0xffffffffull) len = 0xffffffffull;
        const uint64_t pieces = (static_cast<uint64_t>(n_y) + width - 1) / width;
        prm.chunk_begin[g] = n_chunks;
        prm.chunk_len[g] = static_cast<uint32_t>(len);
        prm.prefix_chunks[g] = (prefixes + len - 1) / len;
        prm.y_width[g] = static_cast<uint32_t>(width);
        n_chunks += pieces * prm.prefix_chunks[g];
    }
    prm.chunk_begin[prm.n_groups] = n_chunks;
    const uint64_t my_chunks = n_chunks > static_cast<uint64_t>(part) ? (n_chunks - part + parts - 1) / parts : 0;
    if (my_chunks == 0) {
        *c_max = -1;
        return BZ_OK;
    }
    uint64_t blocks = (my_chunks + kWcBlock - 1) / kWcBlock;
    if (blocks > static_cast<uint64_t>(kWcMaxBlocks)) blocks = kWcMaxBlocks;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    WcResult* dev = static_cast<WcResult*>(workspace);
    const int grid = static_cast<int>(blocks);
    switch ((r + 1) / 2) {
        case 1: launch_tail<1>(tail, grid, s, prm, dev); break;
        case 2: launch_tail<2>(tail, grid, s, prm, dev); break;
        case 3: launch_tail<3>(tail, grid, s, prm, dev); break;
        default: launch_tail<4>(tail, grid, s, prm, dev); break;
    }
    note_launch();
    st = check_launch();
    if (st != BZ_OK) return st;
    return collect_best(dev, static_cast<int>(blocks), K, q, c_max, argmax, s);
}

extern "C" int bz_worst_case(const uint64_t* worker_mask, int K, int f, int r, int q, uint64_t max_subsets,
                             int32_t* c_max, int32_t* argmax, uint64_t* n_subsets, void* workspace,
                             size_t workspace_bytes, void* stream) {
    return worst_case_share(worker_mask, K, f, r, q, 0, 1, max_subsets, c_max, argmax, n_subsets, workspace, workspace_bytes, stream);
}

extern "C" int bz_worst_case_part(const uint64_t* worker_mask, int K, int f, int r, int q, int part, int parts,
                                  uint64_t max_subsets, int32_t* c_max, int32_t* argmax, uint64_t* n_subsets, void* workspace,
                                  size_t workspace_bytes, void* stream) {
    return worst_case_share(worker_mask, K, f, r, q, part, parts, max_subsets, c_max, argmax, n_subsets, workspace, workspace_bytes, stream);
}
