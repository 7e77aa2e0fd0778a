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
int pairdist_i8_stall(int on);
int probe_timeouts(unsigned int* count);          // probe.cu
int* pairdist_status_words(void* ws, int f);      // pairdist.cu

namespace {
std::atomic<uint64_t> g_launches{0};
thread_local char g_cuda_msg[256] = "";

bool is_prime(int n) {
    if (n < 2) return false;
    for (int t = 2; t <= n / t; ++t)
        if (n % t == 0) return false;
    return true;
}

// Arithmetic of the finite field with l = p^k elements (Sec. 4.1.1).  Elements are the integers
// 0 .. l-1 read in base p (digit t = coefficient of x^t).  Products are built digit by digit from the
// top ("multiply the running value by x, reduce, add a times the digit"), with x^k replaced through the
// first monic irreducible polynomial of degree k when the candidates are ordered by their lower
// coefficients read as a base-p number.
class GaloisField {
public:
    bool init(int l) {
        if (l < 2) return false;
        p_ = 2;
        while (l % p_ != 0) ++p_;
        k_ = 0;
        int rest = l;
        while (rest % p_ == 0) {
            rest /= p_;
            ++k_;
        }
        if (rest != 1) return false;
        l_ = l;
        top_ = l / p_;  // p^(k-1): the weight of the leading digit
        if (k_ == 1) {
            low_ = 0;
            return true;
        }
        for (low_ = 0; low_ < l; ++low_)
            if (has_no_factor(low_)) return true;
        return false;
    }
    int add(int a, int b) const {
        int sum = 0, w = 1;
        for (int t = 0; t < k_; ++t, w *= p_, a /= p_, b /= p_) sum += ((a % p_ + b % p_) % p_) * w;
        return sum;
    }
    int scale(int a, int c) const {  // a times the constant c of Z_p
        int out = 0, w = 1;
        for (int t = 0; t < k_; ++t, w *= p_, a /= p_) out += ((a % p_) * c % p_) * w;
        return out;
    }
    int times_x(int a) const {       // a * x with x^k = -(lower part of the modulus)
        const int lead = a / top_;
        const int shifted = (a % top_) * p_;
        return add(shifted, scale(low_, (p_ - lead) % p_));
    }
    int mul(int a, int b) const {
        if (k_ == 1) return static_cast<int>(static_cast<long long>(a) * b % l_);
        int acc = 0;
        for (int w = top_; w >= 1; w /= p_) {
            acc = times_x(acc);
            acc = add(acc, scale(a, (b / w) % p_));
        }
        return acc;
    }

private:
    // is x^k + low(x) free of monic factors of degree 1 .. k/2?  Tested through arithmetic modulo the
    // candidate itself: g divides m iff some nonzero h of degree < k - deg g has g*h = 0 mod m; here simply
    // by evaluating the product of g with every cofactor of the right degree.
    bool has_no_factor(int low) const {
        const int full = l_ + low;  // the monic candidate as a number with k+1 digits
        for (int dg = 1; dg <= k_ / 2; ++dg) {
            int ng = 1, nh = 1;
            for (int t = 0; t < dg; ++t) ng *= p_;
            for (int t = 0; t < k_ - dg; ++t) nh *= p_;
            for (int g = ng; g < 2 * ng; ++g)          // monic of degree dg: leading digit 1
                for (int h = nh; h < 2 * nh; ++h)      // monic of degree k - dg
                    if (plain_product(g, h) == full) return false;
        }
        return true;
    }
    int plain_product(int g, int h) const {  // polynomial product over Z_p without reduction
        int digits_g[16], digits_h[16], out[32] = {0};
        int ng = 0, nh = 0;
        for (; g > 0; g /= p_) digits_g[ng++] = g % p_;
        for (; h > 0; h /= p_) digits_h[nh++] = h % p_;
        for (int t = 0; t < ng; ++t)
            for (int u = 0; u < nh; ++u) out[t + u] = (out[t + u] + digits_g[t] * digits_h[u]) % p_;
        int v = 0;
        for (int t = ng + nh - 2; t >= 0; --t) v = v * p_ + out[t];
        return v;
    }
    int p_ = 0, k_ = 0, l_ = 0, top_ = 0, low_ = 0;
};

}  // namespace

void note_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

thread_local int g_last_path = BZ_PATH_NONE;
void note_path(int path) { g_last_path = path; }

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
    if (l < 2 || l > 46340 || r < 1 || r > l) return BZ_ERR_INVALID_ARG;
    const bool prime = is_prime(l);
    GaloisField field;
    if (!prime && (l > 1024 || !field.init(l))) return BZ_ERR_INVALID_ARG;  // neither a prime nor a (small) prime power
    if (!prime && r > l - 1) return BZ_ERR_INVALID_ARG;  // l - 1 squares exist; r = l only through the bigraph (prime l)
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
                // the column j with alpha*i + j = s
                int j;
                if (prime) {
                    j = static_cast<int>(((s - static_cast<int64_t>(alpha) * i) % l + l) % l);
                } else {
                    const int ai = field.mul(alpha, i);
                    j = 0;
                    while (field.add(ai, j) != s) ++j;
                }
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
    unsigned int a = 0, b = 0, c = 0, p = 0;
    int st = pipeline_timeouts(&a);
    if (st == BZ_OK) st = vote_pairdist_timeouts(&b);
    if (st == BZ_OK) st = pairdist_i8_timeouts(&c);
    if (st == BZ_OK) st = probe_timeouts(&p);
    *count = a + b + c + p;
    return st;
}

extern "C" int bz_pairdist_status(const void* workspace, int f, int32_t* status, void* stream) {
    if (workspace == nullptr || status == nullptr || f < 1) return BZ_ERR_INVALID_ARG;
    if (f > BZ_MAX_F) return BZ_ERR_UNSUPPORTED;
    int words[2] = {0, 0};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(words, pairdist_status_words(const_cast<void*>(workspace), f), sizeof(words),
                                    cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_failed(e);
    *status = (words[0] ? BZ_STATUS_RECOMPUTED : 0) | (words[1] ? BZ_STATUS_STOPPED_EARLY : 0);
    return BZ_OK;
}

extern "C" int bz_debug_stall_pipeline(int on) { return pairdist_i8_stall(on); }

extern "C" int bz_last_path(void) { return g_last_path; }

extern "C" const char* bz_last_cuda_error(void) { return g_cuda_msg; }

extern "C" uint64_t bz_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }
