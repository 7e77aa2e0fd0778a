// CPU oracle for the ByzShield parameter-server aggregation path.
//
// TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, obviously-correct statement of what
// the aggregation path computes, written from the paper's definitions.  It shares no code,
// header, table or helper with the CUDA library and must never be reached from the product
// path; only the test-suite, the smoke check and the benchmark's CPU-baseline leg call it.
//
// Arithmetic: integer / bit-pattern work is exact; every floating-point sum is carried in
// double precision in the index order stated at each function.  The only parallelism is an
// OpenMP "parallel for" over disjoint outputs (coordinates, row pairs, first subset element),
// which cannot change any result.
//
// Parity pins (see tests/test_oracle_*.py): every function below is pinned by values printed in
// the paper, closed forms, brute force on tiny inputs or reductions to library routines, except
// where a header comment says "parity unpinned".
//
//   orc_assign            Algorithm 2 (MOLS placement; prime and prime-power l, Sec. 4.1.1) + Sec. 4.2.1 (Ramanujan Case 2, m = s = l)
//   orc_assign_ramanujan  Sec. 4.2.1 Steps 1-3 and Eq. (7): the array-code matrix B, H = B or B^T
//   orc_vote              Eq. (3): per-file majority over the r returned copies
//   orc_vote_vectorwise   Eq. (3) read on whole vectors (Sec. 2, "Training Protocol")
//   orc_vote_clusters     the same vote with agreement up to a tolerance (Sec. 2; reading of the builder: parity otherwise unpinned by the paper)
//   orc_median            coordinate-wise median of the f winners (Sec. 2 / Sec. 6.1)
//   orc_pairdist ... orc_mean_rows      Krum / Multi-Krum (Sec. 1.2, Sec. 6.1)
//   orc_bulyan_select, orc_trimmed_mean Bulyan (Sec. 1.2 trimmed mean, Sec. 6.1)
//   orc_worst_case        c_max^(q) by exhaustive search (Sec. 5.3.2, Sec. 6.1)
//   orc_model_update      Eq. (1) step on the aggregate, optional momentum (Sec. 6.1)

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

bool is_prime(int n) {
    if (n < 2) return false;
    for (int t = 2; t * t <= n; ++t)
        if (n % t == 0) return false;
    return true;
}

uint32_t bits_of(float x) {
    uint32_t u;
    std::memcpy(&u, &x, 4);
    return u;
}

float float_of(uint32_t u) {
    float x;
    std::memcpy(&x, &u, 4);
    return x;
}

// The finite field with l = p^k elements (Sec. 4.1.1: "pick a prime power l ... addition is over F_l").
// An element is the integer whose base-p digits are the coefficients of a polynomial of degree < k over
// Z_p (digit t = coefficient of x^t).  Sums add coefficients mod p; products are polynomial products
// reduced modulo a monic irreducible polynomial of degree k - the first one when the candidates are
// listed by the integer value of their lower coefficients.  For a prime l (k = 1) this is arithmetic mod l.
struct Field {
    int p = 0, k = 0, l = 0;
    std::vector<int> irr;   // irr[0..k], irr[k] = 1

    std::vector<int> digits(int a, int n) const {
        std::vector<int> c(n, 0);
        for (int t = 0; t < n && a > 0; ++t, a /= p) c[t] = a % p;
        return c;
    }
    int number(const std::vector<int>& c) const {
        int a = 0;
        for (int t = (int)c.size() - 1; t >= 0; --t) a = a * p + c[t];
        return a;
    }
    // remainder of the polynomial c (any degree) on division by the monic polynomial m of degree dm
    std::vector<int> remainder(std::vector<int> c, const std::vector<int>& m, int dm) const {
        for (int t = (int)c.size() - 1; t >= dm; --t) {
            const int q = c[t];
            if (q == 0) continue;
            for (int u = 0; u <= dm; ++u) c[t - dm + u] = ((c[t - dm + u] - q * m[u]) % p + p) % p;
        }
        c.resize(dm);
        return c;
    }
    bool irreducible(const std::vector<int>& m) const {
        // no monic polynomial of degree 1 .. k/2 divides m
        for (int dg = 1; dg <= k / 2; ++dg) {
            int count = 1;
            for (int t = 0; t < dg; ++t) count *= p;
            for (int low = 0; low < count; ++low) {
                std::vector<int> g = digits(low, dg + 1);
                g[dg] = 1;
                std::vector<int> rem = remainder(m, g, dg);
                bool zero = true;
                for (int v : rem) zero = zero && v == 0;
                if (zero) return false;
            }
        }
        return true;
    }
    bool init(int size) {
        if (size < 2) return false;
        int q = 2;
        while (size % q != 0) ++q;   // smallest prime factor
        int kk = 0, rest = size;
        while (rest % q == 0) {
            rest /= q;
            ++kk;
        }
        if (rest != 1) return false;
        p = q;
        k = kk;
        l = size;
        for (int low = 0; low < l; ++low) {
            std::vector<int> m = digits(low, k + 1);
            m[k] = 1;
            if (k == 1 || irreducible(m)) {
                irr = m;
                return true;
            }
        }
        return false;
    }
    int add(int a, int b) const {
        std::vector<int> x = digits(a, k), y = digits(b, k);
        for (int t = 0; t < k; ++t) x[t] = (x[t] + y[t]) % p;
        return number(x);
    }
    int mul(int a, int b) const {
        std::vector<int> x = digits(a, k), y = digits(b, k), c(2 * k - 1 > 0 ? 2 * k - 1 : 1, 0);
        for (int t = 0; t < k; ++t)
            for (int u = 0; u < k; ++u) c[t + u] = (c[t + u] + x[t] * y[u]) % p;
        return number(remainder(c, irr, k));
    }
};

// IEEE-754 total order as an unsigned key: negatives have all bits flipped, non-negatives have
// the sign bit set.  -NaN < -inf < ... < -0 < +0 < ... < +inf < +NaN.
uint32_t order_key(float x) {
    uint32_t u = bits_of(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

float from_order_key(uint32_t k) {
    uint32_t u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
    return float_of(u);
}

// Krum score of row `a` among the rows listed in `rows`: sum of the `nb` smallest squared
// distances from `a` to the other listed rows, added in ascending order of distance.
double krum_score(const double* D, int f, const std::vector<int>& rows, int a, int nb) {
    std::vector<double> dist;
    for (int b : rows)
        if (b != a) dist.push_back(D[(size_t)a * f + b]);
    std::sort(dist.begin(), dist.end());
    double s = 0.0;
    for (int t = 0; t < nb; ++t) s += dist[t];
    return s;
}

}  // namespace

extern "C" {

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

// ---------------------------------------------------------------------------------------------
// Algorithm 2.  Square k uses L_alpha(i, j) = alpha * i + j over F_l (Sec. 4.1.1); the cell
// (i, j) holding symbol s in square k connects file i*l + j to worker k*l + s.
// For r < l the squares are alpha = 1..r (the paper's printed example).  For r = l only l - 1
// MOLS exist; the paper's K = r*l = l^2 cluster is Ramanujan Case 2 with m = s = l, whose
// biadjacency B has block (a, b) = P^(a*b) (Sec. 4.2.1): worker a*l + x holds file b*l + y iff
// a*b + y = x (mod l), i.e. the same rule with alpha = a in {0..l-1}.
// worker_files[K][l] ascending; file_workers[f][r] indexed by class k; worker_mask[K] bit x set
// iff the worker holds file x (only when f <= 64; may be null).
int orc_assign(int l, int r, int32_t* worker_files, int32_t* file_workers, uint64_t* worker_mask) {
    const bool prime = is_prime(l);
    Field F;
    if (!prime && !F.init(l)) return -1;                 // neither a prime nor a prime power
    if (r < 1 || r > l || (!prime && r > l - 1)) return -1;   // Algorithm 2 has l - 1 squares; r = l only via the bigraph (prime l)
    const int K = r * l, f = l * l;
    std::vector<std::vector<int>> held(K);
    for (int k = 0; k < r; ++k) {
        const int alpha = (r == l) ? k : k + 1;
        for (int i = 0; i < l; ++i)
            for (int j = 0; j < l; ++j) {
                const int s = prime ? (alpha * i + j) % l : F.add(F.mul(alpha, i), j);
                const int file = i * l + j, worker = k * l + s;
                held[worker].push_back(file);
                file_workers[file * r + k] = worker;
            }
    }
    for (int u = 0; u < K; ++u) {
        std::sort(held[u].begin(), held[u].end());
        if ((int)held[u].size() != l) return -2;
        for (int t = 0; t < l; ++t) worker_files[u * l + t] = held[u][t];
        if (worker_mask && f <= 64) {
            uint64_t m = 0;
            for (int x : held[u]) m |= (uint64_t)1 << x;
            worker_mask[u] = m;
        }
    }
    return 0;
}

// The field's addition and multiplication tables ([l][l] each), for tests of the field itself.
int orc_field_tables(int l, int32_t* add, int32_t* mul) {
    Field F;
    if (!F.init(l)) return -1;
    for (int a = 0; a < l; ++a)
        for (int b = 0; b < l; ++b) {
            add[a * l + b] = F.add(a, b);
            mul[a * l + b] = F.mul(a, b);
        }
    return 0;
}

// ---------------------------------------------------------------------------------------------
// Sec. 4.2.1, written out: P is the s x s cyclic shift with P[i][j] = 1 iff j = i - 1 (mod s); B is
// the s x m block matrix whose block (a, b) is P^(a*b) (matrix powers by repeated multiplication);
// H = B when m >= s (Case 2: K = s*s workers, f = m*s files) and H = B^T when m < s (Case 1:
// K = m*s workers, f = s*s files), Eq. (7).  Rows of H are workers, columns are files.
// worker_files[K][l] ascending, file_workers[f][r] ascending, worker_mask as in orc_assign.
int orc_assign_ramanujan(int m, int s, int32_t* worker_files, int32_t* file_workers, uint64_t* worker_mask) {
    if (m < 2 || !is_prime(s)) return -1;
    typedef std::vector<std::vector<int>> Mat;
    auto matmul = [&](const Mat& X, const Mat& Y) {
        Mat Z(s, std::vector<int>(s, 0));
        for (int i = 0; i < s; ++i)
            for (int k = 0; k < s; ++k)
                if (X[i][k])
                    for (int j = 0; j < s; ++j) Z[i][j] += X[i][k] * Y[k][j];
        return Z;
    };
    Mat I(s, std::vector<int>(s, 0)), P(s, std::vector<int>(s, 0));
    for (int i = 0; i < s; ++i) {
        I[i][i] = 1;
        P[i][((i - 1) % s + s) % s] = 1;
    }
    const int rows = s * s, cols = m * s;
    std::vector<std::vector<int>> B(rows, std::vector<int>(cols, 0));
    for (int a = 0; a < s; ++a)
        for (int b = 0; b < m; ++b) {
            Mat blk = I;
            for (int t = 0; t < a * b; ++t) blk = matmul(blk, P);
            for (int x = 0; x < s; ++x)
                for (int y = 0; y < s; ++y) B[a * s + x][b * s + y] = blk[x][y];
        }
    const bool case2 = m >= s;
    const int K = case2 ? rows : cols, f = case2 ? cols : rows;
    const int l = case2 ? m : s, r = case2 ? s : m;
    std::vector<int> n_workers(f, 0);
    for (int u = 0; u < K; ++u) {
        int n = 0;
        uint64_t mask = 0;
        for (int x = 0; x < f; ++x) {
            const int h = case2 ? B[u][x] : B[x][u];
            if (h != 0 && h != 1) return -2;
            if (h) {
                if (n >= l || n_workers[x] >= r) return -2;
                worker_files[u * l + n++] = x;
                file_workers[x * r + n_workers[x]++] = u;
                if (f <= 64) mask |= (uint64_t)1 << x;
            }
        }
        if (n != l) return -2;
        if (worker_mask && f <= 64) worker_mask[u] = mask;
    }
    for (int x = 0; x < f; ++x)
        if (n_workers[x] != r) return -2;
    return 0;
}

// ---------------------------------------------------------------------------------------------
// Eq. (3), element by element: for file i and coordinate j the winner is the 32-bit pattern
// that occurs most often among replicas[k][i][j], k = 0..r-1; among equally frequent patterns
// the one whose first occurrence has the lowest k wins.  Equality is on bit patterns.
// replicas is contiguous [r][f][d]; voted is contiguous [f][d].
void orc_vote(const float* replicas, int r, int f, int64_t d, float* voted) {
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < d; ++j)
        for (int i = 0; i < f; ++i) {
            int best_k = 0, best_count = 0;
            for (int k = 0; k < r; ++k) {
                const uint32_t pk = bits_of(replicas[((size_t)k * f + i) * d + j]);
                int count = 0;
                for (int k2 = 0; k2 < r; ++k2)
                    if (bits_of(replicas[((size_t)k2 * f + i) * d + j]) == pk) ++count;
                if (count > best_count) {
                    best_count = count;
                    best_k = k;
                }
            }
            voted[(size_t)i * d + j] = replicas[((size_t)best_k * f + i) * d + j];
        }
}

// Eq. (3) read on whole gradients, as the paper's own implementation did: the copy (as a
// d-vector, exact match) that appears most often wins; ties go to the lowest k.
// winner[i] = index k of the winning copy of file i.
void orc_vote_vectorwise(const float* replicas, int r, int f, int64_t d, int32_t* winner) {
    for (int i = 0; i < f; ++i) {
        int best_k = 0, best_count = 0;
        for (int k = 0; k < r; ++k) {
            const float* vk = replicas + ((size_t)k * f + i) * d;
            int count = 0;
            for (int k2 = 0; k2 < r; ++k2) {
                const float* v2 = replicas + ((size_t)k2 * f + i) * d;
                if (std::memcmp(vk, v2, (size_t)d * 4) == 0) ++count;
            }
            if (count > best_count) {
                best_count = count;
                best_k = k;
            }
        }
        winner[i] = best_k;
    }
}

// The vote on whole vectors with agreement up to a tolerance (Sec. 2, "Training Protocol",
// remarks that copies which differ only by numerical precision can be voted on by grouping the returned
// gradients into clusters; the paper defines no rule - this is the reading taken).  Two copies of a file agree iff
// at every coordinate their bit patterns are equal or |a - b| <= abs_tol + rel_tol * max(|a|, |b|),
// the bound formed in binary32 with one fused multiply-add (the precision the decision is taken in on
// the GPU as well).  The winner is the copy that agrees with the most copies (itself included); ties
// go to the lowest k.  With both tolerances 0 this is orc_vote_vectorwise.
void orc_vote_clusters(const float* replicas, int r, int f, int64_t d, float abs_tol, float rel_tol, int32_t* winner) {
    for (int i = 0; i < f; ++i) {
        int best_k = 0, best_count = 0;
        for (int k = 0; k < r; ++k) {
            const float* vk = replicas + ((size_t)k * f + i) * d;
            int count = 0;
            for (int k2 = 0; k2 < r; ++k2) {
                const float* v2 = replicas + ((size_t)k2 * f + i) * d;
                bool agree = true;
                for (int64_t j = 0; j < d && agree; ++j) {
                    if (bits_of(vk[j]) == bits_of(v2[j])) continue;
                    const float gap = std::fabs(vk[j] - v2[j]);
                    const float bound = std::fmaf(rel_tol, std::fmax(std::fabs(vk[j]), std::fabs(v2[j])), abs_tol);
                    if (!(gap <= bound)) agree = false;
                }
                if (agree) ++count;
            }
            if (count > best_count) {
                best_count = count;
                best_k = k;
            }
        }
        winner[i] = best_k;
    }
}

// ---------------------------------------------------------------------------------------------
// Coordinate-wise median of the f winners: sort the f values of a coordinate by IEEE total
// order and return rank (f-1)/2.  For even f (outside the paper's odd-l configurations) the two
// middle values lo <= hi are combined as 0.5f*lo + 0.5f*hi in single precision.
void orc_median(const float* voted, int f, int64_t d, float* out) {
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < d; ++j) {
        std::vector<uint32_t> key(f);
        for (int i = 0; i < f; ++i) key[i] = order_key(voted[(size_t)i * d + j]);
        std::sort(key.begin(), key.end());
        if (f % 2 == 1) {
            out[j] = from_order_key(key[(f - 1) / 2]);
        } else {
            const float lo = from_order_key(key[f / 2 - 1]), hi = from_order_key(key[f / 2]);
            out[j] = 0.5f * lo + 0.5f * hi;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Squared Euclidean distances between all pairs of rows: D[a][b] = sum_j (v_a[j] - v_b[j])^2,
// each term formed and accumulated in double, j ascending.  D is [f][f], symmetric, zero diagonal.
void orc_pairdist(const float* voted, int f, int64_t d, double* D) {
#pragma omp parallel for schedule(dynamic)
    for (int a = 0; a < f; ++a)
        for (int b = a; b < f; ++b) {
            double s = 0.0;
            if (a != b)
                for (int64_t j = 0; j < d; ++j) {
                    const double t = (double)voted[(size_t)a * d + j] - (double)voted[(size_t)b * d + j];
                    s += t * t;
                }
            D[(size_t)a * f + b] = s;
            D[(size_t)b * f + a] = s;
        }
}

// Krum scores over all f rows assuming c corrupted operands: score[a] = sum of the
// f - c - 2 smallest D[a][b], b != a.
void orc_krum_scores(const double* D, int f, int c, double* score) {
    std::vector<int> rows(f);
    for (int a = 0; a < f; ++a) rows[a] = a;
    for (int a = 0; a < f; ++a) score[a] = krum_score(D, f, rows, a, f - c - 2);
}

// Multi-Krum selection: rank rows by (score, index) ascending, keep the first m (m = 1 is Krum).
// Returns -1 when the operand requirement f >= 2c + 3 (Sec. 6.1) or 1 <= m <= f fails.
int orc_multikrum_select(const double* D, int f, int c, int m, int32_t* selected) {
    if (c < 0 || f < 2 * c + 3 || m < 1 || m > f) return -1;
    std::vector<double> score(f);
    orc_krum_scores(D, f, c, score.data());
    std::vector<int> order(f);
    for (int a = 0; a < f; ++a) order[a] = a;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return score[a] < score[b]; });
    for (int t = 0; t < m; ++t) selected[t] = order[t];
    return 0;
}

// Coordinate-wise mean of the selected rows: double sum in the order of `selected`, divided by
// m in double, rounded once to single.
void orc_mean_rows(const float* voted, int f, int64_t d, const int32_t* selected, int m, float* out) {
    (void)f;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < d; ++j) {
        double s = 0.0;
        for (int t = 0; t < m; ++t) s += (double)voted[(size_t)selected[t] * d + j];
        out[j] = (float)(s / (double)m);
    }
}

// ---------------------------------------------------------------------------------------------
// Bulyan, first stage: theta = f - 2c rows are picked one at a time.  With R the rows not yet
// picked, each pick computes Krum scores inside R with nb = clamp(|R| - c - 2, 1, |R| - 1)
// neighbours (the single remaining row is taken as is) and moves the (score, index)-smallest
// row from R to `selected` (pick order).  Returns -1 unless f >= 4c + 3 (Sec. 6.1).
int orc_bulyan_select(const double* D, int f, int c, int32_t* selected) {
    if (c < 0 || f < 4 * c + 3) return -1;
    const int theta = f - 2 * c;
    std::vector<int> R(f);
    for (int a = 0; a < f; ++a) R[a] = a;
    for (int t = 0; t < theta; ++t) {
        const int n = (int)R.size();
        int pick = 0;
        if (n > 1) {
            int nb = n - c - 2;
            if (nb < 1) nb = 1;
            if (nb > n - 1) nb = n - 1;
            double best = 0.0;
            for (int p = 0; p < n; ++p) {
                const double s = krum_score(D, f, R, R[p], nb);
                if (p == 0 || s < best) {  // R stays ascending, so "<" keeps the lowest index
                    best = s;
                    pick = p;
                }
            }
        }
        selected[t] = R[pick];
        R.erase(R.begin() + pick);
    }
    return 0;
}

// Bulyan, second stage (trimmed mean around the median): per coordinate, sort the theta
// selected values by total order, med = element (theta-1)/2, then grow a window from the median
// position, each step taking the neighbour (below or above) with the smaller |v - med| in
// single precision, ties to the lower side, until it holds beta values; output their mean
// (double sum in ascending sorted order, divided by beta, rounded once).
void orc_trimmed_mean(const float* voted, int f, int64_t d, const int32_t* selected, int theta, int beta,
                      float* out) {
    (void)f;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < d; ++j) {
        std::vector<uint32_t> key(theta);
        for (int t = 0; t < theta; ++t) key[t] = order_key(voted[(size_t)selected[t] * d + j]);
        std::sort(key.begin(), key.end());
        std::vector<float> s(theta);
        for (int t = 0; t < theta; ++t) s[t] = from_order_key(key[t]);
        const int mid = (theta - 1) / 2;
        const float med = s[mid];
        int lo = mid, hi = mid;
        while (hi - lo + 1 < beta) {
            const bool can_lo = lo > 0, can_hi = hi < theta - 1;
            bool take_lo;
            if (can_lo && can_hi) {
                const float dl = std::fabs(s[lo - 1] - med), dh = std::fabs(s[hi + 1] - med);
                take_lo = dl <= dh;
            } else {
                take_lo = can_lo;
            }
            if (take_lo) --lo; else ++hi;
        }
        double sum = 0.0;
        for (int t = lo; t <= hi; ++t) sum += (double)s[t];
        out[j] = (float)(sum / (double)beta);
    }
}

// ---------------------------------------------------------------------------------------------
// c_max^(q): over every q-subset S of the K workers (lexicographic order), count the files with
// at least r' = (r+1)/2 of their r holders inside S; return the maximum and the first subset
// that attains it.  worker_files is [K][l].  n_subsets receives C(K, q).
int orc_worst_case(const int32_t* worker_files, int K, int l, int f, int r, int q, int32_t* c_max,
                   int32_t* argmax, uint64_t* n_subsets) {
    if (q < 0 || q > K || r < 1) return -1;
    const int rp = (r + 1) / 2;
    if (q == 0) {
        *c_max = 0;
        if (n_subsets) *n_subsets = 1;
        return 0;
    }
    const int n_first = K - q + 1;  // possible values of the smallest element
    std::vector<int> best_cnt(n_first, -1);
    std::vector<std::vector<int>> best_set(n_first);
    std::vector<uint64_t> visited(n_first, 0);
#pragma omp parallel for schedule(dynamic)
    for (int first = 0; first < n_first; ++first) {
        std::vector<int> S(q);
        S[0] = first;
        for (int t = 1; t < q; ++t) S[t] = first + t;
        std::vector<int> holders(f);
        while (true) {
            std::fill(holders.begin(), holders.end(), 0);
            for (int t = 0; t < q; ++t)
                for (int e = 0; e < l; ++e) ++holders[worker_files[S[t] * l + e]];
            int cnt = 0;
            for (int x = 0; x < f; ++x)
                if (holders[x] >= rp) ++cnt;
            ++visited[first];
            if (cnt > best_cnt[first]) {
                best_cnt[first] = cnt;
                best_set[first] = S;
            }
            // lexicographic successor with S[0] held fixed
            int t = q - 1;
            while (t >= 1 && S[t] == K - q + t) --t;
            if (t < 1) break;
            ++S[t];
            for (int u = t + 1; u < q; ++u) S[u] = S[u - 1] + 1;
        }
    }
    int best = -1, arg = 0;
    uint64_t total = 0;
    for (int first = 0; first < n_first; ++first) {
        total += visited[first];
        if (best_cnt[first] > best) {
            best = best_cnt[first];
            arg = first;
        }
    }
    *c_max = best;
    if (argmax)
        for (int t = 0; t < q; ++t) argmax[t] = best_set[arg][t];
    if (n_subsets) *n_subsets = total;
    return 0;
}

// Number of files whose majority is held by the given worker set (the quantity c_max maximises).
int orc_count_distorted(const int32_t* file_workers, int f, int r, const int32_t* byz, int q) {
    const int rp = (r + 1) / 2;
    int cnt = 0;
    for (int x = 0; x < f; ++x) {
        int holders = 0;
        for (int k = 0; k < r; ++k)
            for (int t = 0; t < q; ++t)
                if (file_workers[x * r + k] == byz[t]) ++holders;
        if (holders >= rp) ++cnt;
    }
    return cnt;
}

// ---------------------------------------------------------------------------------------------
// Eq. (1) / Algorithm 1, the parameter server's last step: w <- w - eta * g with g the aggregate.
// With a momentum coefficient mu (Sec. 6.1 trains with 0.9; the paper gives no formula, so the
// heavy-ball form of the framework it trained with is taken): v <- mu * v + g, w <- w - eta * v.
// v == null is the plain step of Eq. (1).  w and v are single-precision state; each new value is
// formed in double from the stored singles and rounded once.
void orc_model_update(float* w, float* v, const float* g, int64_t d, float eta, float mu) {
    for (int64_t j = 0; j < d; ++j) {
        double step = static_cast<double>(g[j]);
        if (v != nullptr) {
            v[j] = static_cast<float>(static_cast<double>(mu) * static_cast<double>(v[j]) + static_cast<double>(g[j]));
            step = static_cast<double>(v[j]);
        }
        w[j] = static_cast<float>(static_cast<double>(w[j]) - static_cast<double>(eta) * step);
    }
}

}  // extern "C"
