// Host-only entry points and bookkeeping of libbz: the task assignment (Algorithm 2), workspace
// sizes, status strings.
#include <atomic>
#include <cstdio>
#include <cstring>

#include "bz_common.cuh"

namespace bz {

size_t krum_workspace_bytes(int op, int f);   // krum.cu
size_t worst_case_workspace_bytes();          // worst_case.cu
size_t worst_case_mols_workspace_bytes(int l, int r);  // worst_case_mols.cu
size_t vote_vectorwise_workspace(int f);      // vote_vectorwise.cu
int pipeline_timeouts(unsigned int* count);   // vote_median_tma.cu
int vote_pairdist_timeouts(unsigned int* count);  // vote_pairdist.cu
int pairdist_i8_timeouts(unsigned int* count);    // pairdist_i8.cu

namespace {
std::atomic<uint64_t> g_launches{0};
thread_local char g_cuda_msg[256] = "";

bool is_prime(int n) {
    if (n < 2) return false;
    for (int t = 2; t <= n / t; ++t)
        if (n % t == 0) return false;
    return true;
}
}  // namespace

void note_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

int cuda_failed(cudaError_t e) {
    std::snprintf(g_cuda_msg, sizeof(g_cuda_msg), "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
    return BZ_ERR_CUDA;
}

int check_launch() {
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? BZ_OK : cuda_failed(e);
}

}  // namespace bz

using namespace bz;

extern "C" int bz_assign_mols(int l, int r, int32_t* worker_files, int32_t* file_workers, uint64_t* worker_mask) {
    if (l < 2 || l > 46340 || !is_prime(l) || r < 1 || r > l) return BZ_ERR_INVALID_ARG;
    const int64_t f = static_cast<int64_t>(l) * l;
    if (worker_mask != nullptr && f > 64) return BZ_ERR_INVALID_ARG;
    const int K = r * l;
    if (worker_mask)
        for (int u = 0; u < K; ++u) worker_mask[u] = 0;
    // Parallel class k: slope alpha = k+1 (a Latin square) for r < l, alpha = k for r == l.
    // Worker k*l + s holds the cells (i, j) with alpha*i + j = s (mod l): one per row i, and the
    // file index i*l + j grows with i, so listing rows in order gives the ascending file list.
    for (int k = 0; k < r; ++k) {
        const int alpha = (r == l) ? k : k + 1;
        for (int s = 0; s < l; ++s) {
            const int u = k * l + s;
            for (int i = 0; i < l; ++i) {
                const int j = static_cast<int>(((s - static_cast<int64_t>(alpha) * i) % l + l) % l);
                const int file = i * l + j;
                if (worker_files) worker_files[static_cast<int64_t>(u) * l + i] = file;
                if (file_workers) file_workers[static_cast<int64_t>(file) * r + k] = u;
                if (worker_mask) worker_mask[u] |= 1ull << file;
            }
        }
    }
    return BZ_OK;
}

extern "C" int bz_assign_ramanujan(int m, int s, int32_t* worker_files, int32_t* file_workers, uint64_t* worker_mask) {
    if (m < 2 || s < 2 || s > 46340 || m > 46340 || !is_prime(s)) return BZ_ERR_INVALID_ARG;
    // Block (a, b) of the array-code matrix is the a*b-th power of the cyclic shift: its entry (x, y)
    // is 1 iff y = x - a*b (mod s).  m >= s: H = B, worker a*s + x holds file b*s + y.
    // m < s: H = B^T, worker b*s + y holds file a*s + x.
    const bool case2 = m >= s;
    const int64_t K = case2 ? static_cast<int64_t>(s) * s : static_cast<int64_t>(m) * s;
    const int64_t f = case2 ? static_cast<int64_t>(m) * s : static_cast<int64_t>(s) * s;
    const int l = case2 ? m : s, r = case2 ? s : m;
    if (worker_mask != nullptr && f > 64) return BZ_ERR_INVALID_ARG;
    if (worker_mask)
        for (int64_t u = 0; u < K; ++u) worker_mask[u] = 0;
    for (int a = 0; a < s; ++a)
        for (int b = 0; b < m; ++b) {
            const int shift = static_cast<int>((static_cast<int64_t>(a) * b) % s);
            for (int x = 0; x < s; ++x) {
                const int y = (x - shift + s) % s;
                const int64_t row = static_cast<int64_t>(a) * s + x, col = static_cast<int64_t>(b) * s + y;
                const int64_t worker = case2 ? row : col, file = case2 ? col : row;
                // the class of a worker (a resp. b) and the block index on the file side (b resp. a) order both lists
                const int in_worker = case2 ? b : a, in_file = case2 ? a : b;
                if (worker_files) worker_files[worker * l + in_worker] = static_cast<int32_t>(file);
                if (file_workers) file_workers[file * r + in_file] = static_cast<int32_t>(worker);
                if (worker_mask) worker_mask[worker] |= 1ull << file;
            }
        }
    return BZ_OK;
}

extern "C" size_t bz_workspace_bytes(int op, int r, int f, int64_t d, int c, int m) {
    (void)c;
    (void)m;
    if (f < 1 || f > BZ_MAX_F) return 0;
    switch (op) {
        case BZ_OP_PAIRDIST:
        case BZ_OP_MULTIKRUM:
        case BZ_OP_BULYAN: return krum_workspace_bytes(op, f);
        case BZ_OP_WORST_CASE: return worst_case_workspace_bytes();
        case BZ_OP_VOTE_VECTORWISE: return vote_vectorwise_workspace(f);
        case BZ_OP_WORST_CASE_MOLS: {
            int l = 2;
            while (l * l < f) ++l;
            if (l * l != f || l > 7 || r < 1 || r > l) return 0;
            return worst_case_mols_workspace_bytes(l, r);
        }
        case BZ_OP_VOTE_MEDIAN_HOST: {
            if (r < 1 || d < 0) return 0;
            // smallest useful slab: 64K coordinates (or all of them) of r*f rows plus the output row
            int64_t S = d < 65536 ? (d + 63) / 64 * 64 : 65536;
            if (S < 64) S = 64;
            return round_up((static_cast<size_t>(r) * f + 1) * S * sizeof(float), 256);
        }
        default: return 0;
    }
}

extern "C" const char* bz_status_string(int status) {
    switch (status) {
        case BZ_OK: return "ok";
        case BZ_ERR_INVALID_ARG: return "invalid argument";
        case BZ_ERR_UNSUPPORTED: return "shape outside the compiled limits";
        case BZ_ERR_PRECONDITION: return "operand-count precondition of the aggregator not met";
        case BZ_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case BZ_ERR_BUDGET: return "number of subsets exceeds the budget";
        case BZ_ERR_CUDA: return "CUDA runtime error";
        case BZ_ERR_STATIC_LIMIT: return "shape needs more scratch than the library's built-in array holds";
        default: return "unknown status";
    }
}

extern "C" int bz_pipeline_timeouts(unsigned int* count) {
    if (count == nullptr) return BZ_ERR_INVALID_ARG;
    unsigned int a = 0, b = 0, c = 0;
    int st = pipeline_timeouts(&a);
    if (st == BZ_OK) st = vote_pairdist_timeouts(&b);
    if (st == BZ_OK) st = pairdist_i8_timeouts(&c);
    *count = a + b + c;
    return st;
}

extern "C" const char* bz_last_cuda_error(void) { return g_cuda_msg; }

extern "C" uint64_t bz_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }
