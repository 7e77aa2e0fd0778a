// Exhaustive worst-case search (Sec. 5.3.2, Sec. 6.1) for the MOLS / Ramanujan Case 2 placements of
// Algorithm 2, cut down by the symmetry of the design.
//
// Worker k*l + s holds the files (i, j) with alpha_k*i + j = s (mod l).  Moving every file by
// (i, j) -> (i + a, j + b) maps worker (k, s) to (k, s + alpha_k*a + b): the l*l translations are
// automorphisms of the bigraph, they keep each parallel class and shift its symbols cyclically, and
// the number of distorted files is the same for a set of workers and for its image.  So one set per
// orbit is enough.  The lexicographically first maximiser is the smallest set of its own orbit,
// which pins down its shape: written class by class as symbol sets S_0 .. S_{r-1}, the first class
// that is neither empty nor full has the smallest sorted list among its l cyclic shifts (all shifts
// can be reached), and - of the l translations that then remain, which shift every other class by a
// different amount - so has the second such class.  The search visits exactly the sets of that
// shape: one per orbit, the wanted maximiser among them.
//
// A class adds at most one holder to a file, so a whole class is added to the bit-sliced counts
// with one ripple-carry add of the union of its workers' masks; a subset costs r such adds instead
// of q.  Sets are enumerated by composition (how many workers per class), then by the patterns of
// the first r-2 classes (one "head" per thread and step, advanced like an odometer), then by two
// nested loops over the patterns of the last two classes.
#include <vector>

#include "worst_case_common.cuh"

namespace bz {

namespace {

constexpr int kMaxL = 7;     // l*l <= 64 files
constexpr int kMaxR = 7;
constexpr int kSlots = 192;  // 2^7 patterns grouped by size, then the canonical ones grouped by size
constexpr int kEntry = 8;    // per composition: one (first slot << 16 | count) word per class

struct MolsArgs {
    const uint64_t* unions;   // [r][kSlots] union of the file masks of the pattern's workers
    const uint8_t* patterns;  // [kSlots] pattern of each slot, symbol s at bit l-1-s
    const uint64_t* cum;      // [n_comp + 1] heads before each composition
    const uint32_t* entries;  // [n_comp][kEntry]
    uint64_t total_heads;
    uint32_t heads_per_chunk;
    uint32_t part, parts;     // this launch takes the chunks whose index is part modulo parts
    int n_comp, l, r;
};

template <int RP>
__global__ void __launch_bounds__(kWcBlock) worst_case_mols_kernel(const MolsArgs a, WcResult* __restrict__ results) {
    __shared__ uint64_t s_union[kMaxR * kSlots];
    __shared__ uint8_t s_pat[kSlots];
    __shared__ int32_t s_cnt[kWcBlock];
    __shared__ uint64_t s_mem[kWcBlock];
    for (int i = threadIdx.x; i < a.r * kSlots; i += blockDim.x) s_union[i] = a.unions[i];
    for (int i = threadIdx.x; i < kSlots; i += blockDim.x) s_pat[i] = a.patterns[i];
    __syncthreads();

    const int l = a.l, H = a.r - 2;  // H head classes, then classes H and H+1 in the nested loops
    const int shift_a = 64 - (H + 1) * l, shift_b = 64 - (H + 2) * l;
    Best best{-1, 0};
    uint32_t e[kMaxR];
    int dig[kMaxR];
    Planes st[kMaxR];
    uint64_t mem[kMaxR];
    st[0] = Planes{0, 0, 0};
    mem[0] = 0;

    const uint64_t n_chunks = (a.total_heads + a.heads_per_chunk - 1) / a.heads_per_chunk;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    for (uint64_t unit = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x;; unit += stride) {
        const uint64_t chunk = a.part + a.parts * unit;
        if (chunk >= n_chunks) break;
        uint64_t head = chunk * a.heads_per_chunk;
        const uint64_t end = head + a.heads_per_chunk < a.total_heads ? head + a.heads_per_chunk : a.total_heads;
        // composition holding this head: the last c with cum[c] <= head
        int c = 0;
        for (int hi = a.n_comp; hi - c > 1;) {
            const int mid = (c + hi) >> 1;
            if (a.cum[mid] <= head)
                c = mid;
            else
                hi = mid;
        }
        for (int k = 0; k < a.r; ++k) e[k] = a.entries[static_cast<size_t>(c) * kEntry + k];
        uint64_t idx = head - a.cum[c];
        for (int k = H - 1; k >= 0; --k) {  // class 0 is the most significant digit
            const uint32_t n = e[k] & 0xffffu;
            dig[k] = static_cast<int>(idx % n);
            idx /= n;
        }
        int first_changed = 0;
        while (true) {
            for (int k = first_changed; k < H; ++k) {
                const int slot = static_cast<int>(e[k] >> 16) + dig[k];
                st[k + 1] = add_mask(st[k], s_union[k * kSlots + slot]);
                mem[k + 1] = mem[k] | (static_cast<uint64_t>(s_pat[slot]) << (64 - (k + 1) * l));
            }
            const int off_a = static_cast<int>(e[H] >> 16), n_a = static_cast<int>(e[H] & 0xffffu);
            const int off_b = static_cast<int>(e[H + 1] >> 16), n_b = static_cast<int>(e[H + 1] & 0xffffu);
            const uint64_t* ua = s_union + H * kSlots + off_a;
            const uint64_t* ub = s_union + (H + 1) * kSlots + off_b;
            for (int ia = 0; ia < n_a; ++ia) {
                const Planes sa = add_mask(st[H], ua[ia]);
                // the last class adds at most one holder per file: it distorts the files one holder short
                const int base = count_at_least<RP>(sa);
                const uint64_t tip = one_short<RP>(sa);
                for (int ib = 0; ib < n_b; ++ib) {
                    const int cnt = base + __popcll(ub[ib] & tip);
                    if (cnt >= best.cnt)
                        offer(best, cnt,
                              mem[H] | (static_cast<uint64_t>(s_pat[off_a + ia]) << shift_a) |
                                  (static_cast<uint64_t>(s_pat[off_b + ib]) << shift_b));
                }
            }
            if (++head == end) break;
            int k = H - 1;
            while (k >= 0 && ++dig[k] == static_cast<int>(e[k] & 0xffffu)) dig[k--] = 0;
            if (k < 0) {  // the composition is exhausted; head < total_heads, so another one follows
                ++c;
                for (int t = 0; t < a.r; ++t) e[t] = a.entries[static_cast<size_t>(c) * kEntry + t];
                k = 0;
            }
            first_changed = k;
        }
    }
    block_best(best, s_cnt, s_mem, results);
}

// ---- host side: patterns, canonical patterns, compositions -----------------------------------------

struct Tables {
    int l = 0;
    uint8_t pattern[kSlots] = {};
    int full_off[kMaxL + 1] = {}, full_cnt[kMaxL + 1] = {};
    int canon_off[kMaxL + 1] = {}, canon_cnt[kMaxL + 1] = {};
};

int popcount8(unsigned p) {
    int n = 0;
    for (; p; p &= p - 1) ++n;
    return n;
}

// symbol s sits at bit l-1-s: of two patterns of one size the larger word has the smaller sorted list
unsigned shifted_pattern(unsigned p, int t, int l) {
    unsigned out = 0;
    for (int s = 0; s < l; ++s)
        if (p & (1u << (l - 1 - s))) out |= 1u << (l - 1 - (s + t) % l);
    return out;
}

Tables make_tables(int l) {
    Tables T;
    T.l = l;
    int slot = 0;
    for (int pass = 0; pass < 2; ++pass)  // 0: every pattern, 1: the smallest of each cyclic class
        for (int m = 0; m <= l; ++m) {
            (pass == 0 ? T.full_off : T.canon_off)[m] = slot;
            for (int p = (1 << l) - 1; p >= 0; --p) {  // descending word = ascending sorted list
                if (popcount8(p) != m) continue;
                if (pass == 1) {
                    bool smallest = true;
                    for (int t = 1; t < l; ++t) smallest = smallest && shifted_pattern(p, t, l) <= static_cast<unsigned>(p);
                    if (!smallest) continue;
                }
                T.pattern[slot++] = static_cast<uint8_t>(p);
            }
            (pass == 0 ? T.full_cnt : T.canon_cnt)[m] = slot - (pass == 0 ? T.full_off : T.canon_off)[m];
        }
    return T;
}

struct Compositions {
    std::vector<uint64_t> cum;      // heads before each composition, then the total
    std::vector<uint32_t> entries;  // kEntry words per composition
    uint64_t orbits = 0;
};

// Every (m_0..m_{r-1}) with 0 <= m_k <= l and sum q.  The first two classes that are neither empty
// nor full draw from the canonical patterns, the others from all patterns of their size.
Compositions make_compositions(const Tables& T, int r, int q, bool keep_tables) {
    Compositions C;
    const int l = T.l;
    int m[kMaxR] = {};
    uint64_t heads_total = 0;
    // odometer over m_0..m_{r-2}; the last class takes what is left
    while (true) {
        int used = 0;
        for (int k = 0; k < r - 1; ++k) used += m[k];
        const int last = q - used;
        if (last >= 0 && last <= l) {
            m[r - 1] = last;
            int partial_seen = 0;
            uint64_t heads = 1, subsets = 1;
            uint32_t entry[kEntry] = {};
            for (int k = 0; k < r; ++k) {
                const bool partial = m[k] > 0 && m[k] < l;
                const bool canon = partial && partial_seen < 2;
                if (partial) ++partial_seen;
                const int off = canon ? T.canon_off[m[k]] : T.full_off[m[k]];
                const int cnt = canon ? T.canon_cnt[m[k]] : T.full_cnt[m[k]];
                entry[k] = (static_cast<uint32_t>(off) << 16) | static_cast<uint32_t>(cnt);
                subsets *= static_cast<uint64_t>(cnt);
                if (k < r - 2) heads *= static_cast<uint64_t>(cnt);
            }
            if (keep_tables) {
                C.cum.push_back(heads_total);
                C.entries.insert(C.entries.end(), entry, entry + kEntry);
            }
            heads_total += heads;
            C.orbits += subsets;
        }
        int k = r - 2;
        while (k >= 0 && ++m[k] > l) m[k--] = 0;
        if (k < 0) break;
    }
    if (keep_tables) C.cum.push_back(heads_total);
    return C;
}

bool is_prime_small(int n) {
    if (n < 2) return false;
    for (int t = 2; t * t <= n; ++t)
        if (n % t == 0) return false;
    return true;
}

int validate_mols(int l, int r, int q) {
    if (l < 2 || !is_prime_small(l) || r < 1 || r > l || (r % 2) == 0 || q < 0 || q > r * l) return BZ_ERR_INVALID_ARG;
    if (l > kMaxL || r > kMaxR) return BZ_ERR_UNSUPPORTED;
    return BZ_OK;
}

size_t pad256(size_t x) { return round_up(x, 256); }

}  // namespace

// results | unions | patterns | cum | entries, for the largest number of compositions any q can have
size_t worst_case_mols_workspace_bytes(int l, int r) {
    size_t comps = 1;
    for (int k = 0; k < r - 1; ++k) comps *= static_cast<size_t>(l + 1);
    return pad256(sizeof(WcResult) * kWcMaxBlocks) + pad256(sizeof(uint64_t) * kMaxR * kSlots) + pad256(kSlots) +
           pad256(sizeof(uint64_t) * (comps + 1)) + pad256(sizeof(uint32_t) * kEntry * comps);
}

}  // namespace bz

using namespace bz;

extern "C" int bz_mols_orbit_count(int l, int r, int q, uint64_t* n_orbits) {
    if (n_orbits == nullptr) return BZ_ERR_INVALID_ARG;
    const int st = validate_mols(l, r, q);
    if (st != BZ_OK) return st;
    if (r < 3) return BZ_ERR_UNSUPPORTED;
    *n_orbits = make_compositions(make_tables(l), r, q, false).orbits;
    return BZ_OK;
}

// Share `part` of `parts` of the search (the whole search: 0 of 1); a share without a chunk reports c_max = -1.
static int worst_case_mols_share(int l, int r, int q, int part, int parts, uint64_t max_subsets, int32_t* c_max, int32_t* argmax,
                                 uint64_t* n_orbits, void* workspace, size_t workspace_bytes, void* stream) {
    if (c_max == nullptr) return BZ_ERR_INVALID_ARG;
    if (parts < 1 || part < 0 || part >= parts) return BZ_ERR_INVALID_ARG;
    int st = validate_mols(l, r, q);
    if (st != BZ_OK) return st;
    if (r < 3) return BZ_ERR_UNSUPPORTED;
    if (workspace == nullptr || !aligned256(workspace) || workspace_bytes < worst_case_mols_workspace_bytes(l, r))
        return BZ_ERR_WORKSPACE;
    const int K = r * l;
    uint64_t mask[kMaxL * kMaxR];
    st = bz_assign_mols(l, r, nullptr, nullptr, mask);
    if (st != BZ_OK) return st;
    const Tables T = make_tables(l);
    const Compositions C = make_compositions(T, r, q, true);
    if (max_subsets != 0 && C.orbits > max_subsets) return BZ_ERR_BUDGET;
    if (n_orbits) *n_orbits = C.orbits;
    if (q == 0) {
        *c_max = part == 0 ? 0 : -1;  // the one (empty) set belongs to the first share
        return BZ_OK;
    }
    // union of the file masks of each pattern's workers, per class
    std::vector<uint64_t> unions(static_cast<size_t>(kMaxR) * kSlots, 0);
    for (int k = 0; k < r; ++k)
        for (int slot = 0; slot < kSlots; ++slot)
            for (int s = 0; s < l; ++s)
                if (T.pattern[slot] & (1u << (l - 1 - s))) unions[static_cast<size_t>(k) * kSlots + slot] |= mask[k * l + s];

    const int n_comp = static_cast<int>(C.cum.size()) - 1;
    unsigned char* base = static_cast<unsigned char*>(workspace);
    WcResult* dev_results = reinterpret_cast<WcResult*>(base);
    size_t at = pad256(sizeof(WcResult) * kWcMaxBlocks);
    uint64_t* dev_unions = reinterpret_cast<uint64_t*>(base + at);
    at += pad256(sizeof(uint64_t) * kMaxR * kSlots);
    uint8_t* dev_patterns = reinterpret_cast<uint8_t*>(base + at);
    at += pad256(kSlots);
    uint64_t* dev_cum = reinterpret_cast<uint64_t*>(base + at);
    at += pad256(sizeof(uint64_t) * (C.cum.size()));
    uint32_t* dev_entries = reinterpret_cast<uint32_t*>(base + at);
    at += pad256(sizeof(uint32_t) * C.entries.size());
    if (at > workspace_bytes) return BZ_ERR_WORKSPACE;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(dev_unions, unions.data(), sizeof(uint64_t) * unions.size(), cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dev_patterns, T.pattern, kSlots, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(dev_cum, C.cum.data(), sizeof(uint64_t) * C.cum.size(), cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(dev_entries, C.entries.data(), sizeof(uint32_t) * C.entries.size(), cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) {
        cudaStreamSynchronize(s);  // the host vectors go out of scope
        return cuda_failed(e);
    }

    MolsArgs a;
    a.unions = dev_unions;
    a.patterns = dev_patterns;
    a.cum = dev_cum;
    a.entries = dev_entries;
    a.total_heads = C.cum.back();
    a.n_comp = n_comp;
    a.l = l;
    a.r = r;
    // a few chunks per thread when there is enough work, one head per chunk otherwise
    uint64_t per_chunk = a.total_heads / (static_cast<uint64_t>(kWcMaxBlocks) * kWcBlock * 4);
    if (per_chunk < 1) per_chunk = 1;
    if (per_chunk > 64) per_chunk = 64;
    a.heads_per_chunk = static_cast<uint32_t>(per_chunk);
    a.part = static_cast<uint32_t>(part);
    a.parts = static_cast<uint32_t>(parts);
    const uint64_t n_chunks = (a.total_heads + per_chunk - 1) / per_chunk;
    const uint64_t my_chunks = n_chunks > static_cast<uint64_t>(part) ? (n_chunks - part + parts - 1) / parts : 0;
    if (my_chunks == 0) {
        cudaStreamSynchronize(s);  // the host vectors of the copies above go out of scope
        *c_max = -1;
        return BZ_OK;
    }
    uint64_t blocks = (my_chunks + kWcBlock - 1) / kWcBlock;
    if (blocks > static_cast<uint64_t>(kWcMaxBlocks)) blocks = kWcMaxBlocks;
    const int grid = static_cast<int>(blocks);
    switch ((r + 1) / 2) {
        case 2: worst_case_mols_kernel<2><<<grid, kWcBlock, 0, s>>>(a, dev_results); break;
        case 3: worst_case_mols_kernel<3><<<grid, kWcBlock, 0, s>>>(a, dev_results); break;
        default: worst_case_mols_kernel<4><<<grid, kWcBlock, 0, s>>>(a, dev_results); break;
    }
    note_launch();
    st = check_launch();
    if (st != BZ_OK) {
        cudaStreamSynchronize(s);
        return st;
    }
    return collect_best(dev_results, grid, K, q, c_max, argmax, s);  // waits for the stream: the vectors may go
}

extern "C" int bz_worst_case_mols(int l, int r, int q, uint64_t max_subsets, int32_t* c_max, int32_t* argmax,
                                  uint64_t* n_orbits, void* workspace, size_t workspace_bytes, void* stream) {
    return worst_case_mols_share(l, r, q, 0, 1, max_subsets, c_max, argmax, n_orbits, workspace, workspace_bytes, stream);
}

extern "C" int bz_worst_case_mols_part(int l, int r, int q, int part, int parts, uint64_t max_subsets, int32_t* c_max,
                                       int32_t* argmax, uint64_t* n_orbits, void* workspace, size_t workspace_bytes, void* stream) {
    return worst_case_mols_share(l, r, q, part, parts, max_subsets, c_max, argmax, n_orbits, workspace, workspace_bytes, stream);
}
