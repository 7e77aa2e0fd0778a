/*
 * libbz - parameter-server aggregation of ByzShield (Konstantinidis & Ramamoorthy, MLSys 2021)
 * on one NVIDIA B200 (sm_100a).  C ABI: plain pointers and sizes, no framework types.
 *
 * The library covers the per-round work of the parameter server once the K = r*l workers have
 * reported one gradient for each of their l files: the majority vote over the r copies of every
 * file gradient (Eq. 3, Algorithm 1), the robust aggregation of the f winners (coordinate-wise
 * median in ByzShield, Sec. 2 and Sec. 6.1; Multi-Krum and Bulyan as the alternatives named in
 * Sec. 6.1 and Sec. 7), the task assignment that decides which r workers hold a file
 * (Algorithm 2, Sec. 4.2.1) and the exhaustive worst-case count c_max^(q) (Sec. 5.3.2).
 *
 * Conventions
 *   - "device" pointers are CUDA global-memory addresses of the current device; "host" pointers
 *     are ordinary process memory.  The caller owns every buffer.  The library never allocates
 *     or frees device memory; scratch space is a caller-provided device workspace whose size
 *     bz_workspace_bytes() reports.  Device state that outlives a call is limited to what is part
 *     of the library image: four counters of expired waits (bz_pipeline_timeouts), the switch of
 *     bz_debug_stall_pipeline and the built-in array of bz_pairdist_static.  None of it
 *     influences a result.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls with
 *     device outputs only enqueue work on that stream and return; outputs are valid once the
 *     caller has synchronised it.  Calls with host outputs synchronise the stream themselves.
 *   - Leading dimensions (ld_*) are in elements.  Gradients are IEEE binary32.  Row layout:
 *     replicas[k][i][j] sits at replicas + k*ld_replica + i*ld_file + j, with k the parallel
 *     class (Latin square) of the worker that sent the copy, i the file, j the coordinate.
 *     The fastest kernels need 16-byte aligned bases and leading dimensions that are
 *     multiples of 4; 8-byte alignment with even leading dimensions still gets 64-bit loads;
 *     anything else takes a slower scalar path, never an error.
 *   - Every function returns BZ_OK or a negative status.  Arguments are validated on the host
 *     before anything is launched; on a non-zero status no output has been written and nothing
 *     has been enqueued (BZ_ERR_CUDA excepted: the runtime's message is kept for
 *     bz_last_cuda_error()).  Nothing aborts or throws.
 *   - Limits: r odd, 1 <= r <= BZ_MAX_R; 1 <= f <= BZ_MAX_F; d >= 0 (d == 0 is a successful no-op).
 */
#ifndef BZ_H_
#define BZ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BZ_OK 0
#define BZ_ERR_INVALID_ARG (-1)  /* null pointer, size out of range, r even, l no prime power, r > l */
#define BZ_ERR_UNSUPPORTED (-2)  /* a shape outside the compiled limits                              */
#define BZ_ERR_PRECONDITION (-3) /* f < 2c+3 (Multi-Krum) or f < 4c+3 (Bulyan), m outside [1, f]     */
#define BZ_ERR_WORKSPACE (-4)    /* workspace missing, misaligned (256 B) or too small               */
#define BZ_ERR_BUDGET (-5)       /* C(K, q) exceeds max_subsets                                      */
#define BZ_ERR_CUDA (-6)         /* a CUDA runtime call or launch failed                             */
#define BZ_ERR_STATIC_LIMIT (-7) /* the shape needs more scratch than the built-in array holds       */

#define BZ_MAX_R 15
#define BZ_MAX_F 128

/* operations known to bz_workspace_bytes() */
#define BZ_OP_PAIRDIST 1
#define BZ_OP_MULTIKRUM 2
#define BZ_OP_BULYAN 3
#define BZ_OP_WORST_CASE 4
#define BZ_OP_VOTE_MEDIAN_HOST 5
#define BZ_OP_WORST_CASE_MOLS 6
#define BZ_OP_VOTE_VECTORWISE 7

/*
 * Task assignment (Algorithm 2; Sec. 4.1.1 for the squares L_alpha(i,j) = alpha*i + j over F_l).
 * Square k = 0..r-1 uses alpha = k+1 when r < l.  When r == l the l parallel classes are those of
 * the Ramanujan Case 2 graph with m = s = l (Sec. 4.2.1), i.e. alpha = k.  File i*l + j is given
 * to worker k*l + L(i, j).  Host only, synchronous.
 *   l              a prime with r in [1, l], or a prime power p^k <= 1024 with r in [1, l-1]: then
 *                  F_l is the field of polynomials over Z_p modulo the first monic irreducible
 *                  polynomial of degree k (candidates ordered by their lower coefficients read as
 *                  a base-p number), element = integer whose base-p digits are the coefficients
 *   worker_files   host, int32 [r*l][l]: files of each worker, ascending        (may be NULL)
 *   file_workers   host, int32 [l*l][r]: holder of each file in class k         (may be NULL)
 *   worker_mask    host, uint64 [r*l]: bit x set iff the worker holds file x; requires l*l <= 64
 *                  (may be NULL; BZ_ERR_INVALID_ARG if non-NULL and l*l > 64)
 */
int bz_assign_mols(int l, int r, int32_t* worker_files, int32_t* file_workers, uint64_t* worker_mask);

/*
 * Task assignment from the Ramanujan bigraph of Sec. 4.2.1 (array-code matrix B whose block (a, b)
 * is the a*b-th power of the s x s cyclic shift; H = B for m >= s, H = B^T for m < s).  Cluster
 * shape per Eq. (7): (K, f, l, r) = (m*s, s*s, s, m) if m < s ("Case 1"), (s*s, m*s, m, s) otherwise
 * ("Case 2"); m = s gives the same tables as bz_assign_mols(s, s).  Host only, synchronous.
 *   m >= 2; s prime
 *   worker_files   host, int32 [K][l] ascending            (may be NULL)
 *   file_workers   host, int32 [f][r] ascending            (may be NULL)
 *   worker_mask    host, uint64 [K]; requires f <= 64      (may be NULL)
 */
int bz_assign_ramanujan(int m, int s, int32_t* worker_files, int32_t* file_workers, uint64_t* worker_mask);

/*
 * Majority vote (Eq. 3; Algorithm 1, the loop over files), element by element: voted[i][j] is
 * the 32-bit pattern that occurs most often among replicas[0..r-1][i][j]; among equally frequent
 * patterns the one first seen at the lowest k wins.  Equality is bitwise (+0 != -0, NaNs are
 * equal only with equal payloads).  For colluding attackers this equals the whole-vector vote
 * the paper describes; r odd rules out two-way ties (Sec. 2).
 *   replicas  device, [r][f][d] with ld_file, ld_replica;  voted  device, [f][d] with ld_voted.
 *   voted must not overlap replicas.
 * Two kernels: one on 128-/64-/32-bit register loads (any layout), and - for (r, f) in {3,5}x{25,49} and
 * (7,49), replicas 16-byte aligned with ld_file, ld_replica multiples of 4 - the fused kernel's staged
 * loads with the winners stored directly (any voted layout).  The second is the default from r = 5 up,
 * where it is the faster one; BZ_VOTE_PATH=staged / =registers (environment, read at every call) forces
 * one of them.  Its bounded waits are counted by bz_pipeline_timeouts like the fused kernel's.
 */
int bz_vote(const float* replicas, int r, int f, int64_t d, int64_t ld_file, int64_t ld_replica, float* voted,
            int64_t ld_voted, void* stream);

/*
 * Coordinate-wise median of the f voted gradients (Sec. 2, Sec. 6.1): out[j] is the element of
 * rank (f-1)/2 of voted[0..f-1][j] under the IEEE total order (-NaN < -inf < ... < -0 < +0 < ...
 * < +inf < +NaN).  For even f the two middle values lo <= hi give 0.5f*lo + 0.5f*hi.
 *   voted device [f][d] with ld;  out device [d].
 */
int bz_median(const float* voted, int f, int64_t d, int64_t ld, float* out, void* stream);

/*
 * ByzShield's aggregation in one pass: bz_median(bz_vote(replicas)) without materialising the
 * voted gradients.  Reads 4*r*f bytes and writes 4 bytes per coordinate.
 * The staged kernel behind this call (and behind bz_median and bz_vote_median_update) bounds its
 * waits; should one run out, the kernel stops and part of `out` (of w and velocity) is left
 * unwritten while the call has long returned BZ_OK.  bz_pipeline_timeouts() is how a caller
 * learns of it: the counter has moved.  It never has on a healthy device.
 */
int bz_vote_median(const float* replicas, int r, int f, int64_t d, int64_t ld_file, int64_t ld_replica,
                   float* out, void* stream);

/*
 * bz_vote_median followed by the parameter server's model update (Eq. 1, last step of Algorithm 1)
 * in the same pass, so the aggregate never makes a round trip through memory:
 *     velocity == NULL:  w[j] <- w[j] - eta * g[j]
 *     otherwise:         velocity[j] <- mu * velocity[j] + g[j];  w[j] <- w[j] - eta * velocity[j]
 * with g the coordinate-wise median of the voted gradients (bit-identical to bz_vote_median's out).
 * The momentum form is the heavy-ball one (Sec. 6.1 trains with mu = 0.9 and gives no formula).
 * Each assignment is one fused multiply-add in binary32.
 *   w, velocity  device [d], read and written in place; velocity may be NULL.  Neither may
 *                overlap replicas or out.
 *   out          device [d] or NULL: where non-NULL the aggregate is written as well.
 * Errors as bz_vote_median; BZ_ERR_INVALID_ARG when w is NULL and d > 0.
 */
int bz_vote_median_update(const float* replicas, int r, int f, int64_t d, int64_t ld_file, int64_t ld_replica,
                          float* w, float* velocity, float eta, float mu, float* out, void* stream);

/*
 * The same update from an aggregate g[d] already in device memory (for the Multi-Krum and Bulyan
 * outputs).  g must not overlap w or velocity.
 */
int bz_model_update(const float* g, int64_t d, float* w, float* velocity, float eta, float mu, void* stream);

/*
 * bz_vote_median and bz_vote for copies that do not sit in one strided array (Algorithm 1: the
 * parameter server receives, from each of the K workers, the l gradients of that worker's files -
 * K separate buffers).  rows is a DEVICE table of r*f device pointers: entry k*f + i is copy k of
 * file i, i.e. the gradient worker file_workers[i][k] returned for file i, d floats.  Results are
 * those of bz_vote_median / bz_vote on the same values.  128-bit loads are used when every row
 * (and the output) is 16-byte aligned, which the kernels check themselves; any alignment works.
 *   out    device [d];   voted  device [f][d] with ld_voted.
 */
int bz_vote_median_rows(const float* const* rows, int r, int f, int64_t d, float* out, void* stream);
int bz_vote_rows(const float* const* rows, int r, int f, int64_t d, float* voted, int64_t ld_voted, void* stream);

/*
 * Eq. (3) as the paper states it (Sec. 2, "Training Protocol"): the vote on WHOLE gradients.  For
 * every file the copy whose complete vector (exact match on bit patterns) occurs most often among
 * the file's r copies wins; among equally frequent vectors the one whose first copy has the lowest
 * k.  bz_vote applies the same rule coordinate by coordinate; the two give the same rows whenever
 * a majority of a file's copies is identical (always, with at most r' - 1 Byzantine holders, and
 * whenever the attackers collude).  They differ only when no vector has a majority.
 *   replicas, ld_file, ld_replica as bz_vote.
 *   voted   device [f][d] with ld_voted: the winning copies (may be NULL if only `winner` is wanted).
 *   winner  device int32 [f]: index k of the winning copy of each file (may be NULL).
 *   workspace device, bz_workspace_bytes(BZ_OP_VOTE_VECTORWISE, r, f, d, 0, 0) bytes, 256-byte aligned.
 */
int bz_vote_vectorwise(const float* replicas, int r, int f, int64_t d, int64_t ld_file, int64_t ld_replica, float* voted,
                       int64_t ld_voted, int32_t* winner, void* workspace, size_t workspace_bytes, void* stream);

/*
 * bz_vote_vectorwise with agreement up to a tolerance, for clusters whose honest workers do not return
 * bit-identical gradients (Sec. 2, "Training Protocol", remarks that copies differing only by
 * numerical precision can be voted on by grouping them into clusters; the paper gives no
 * rule, this one is the library's).  Two copies of a file agree iff at every coordinate their bit
 * patterns are equal or |a - b| <= abs_tol + rel_tol * max(|a|, |b|) (binary32, one fused
 * multiply-add for the bound; a NaN agrees only with its own bit pattern).  The winner is the copy
 * that agrees with the most copies of its file, itself included (agreement need not be transitive);
 * ties go to the lowest k.  The winning COPY is returned, not an average.  abs_tol = rel_tol = 0
 * is bz_vote_vectorwise.  BZ_ERR_INVALID_ARG for negative or NaN tolerances.
 */
int bz_vote_clusters(const float* replicas, int r, int f, int64_t d, int64_t ld_file, int64_t ld_replica, float abs_tol,
                     float rel_tol, float* voted, int64_t ld_voted, int32_t* winner, void* workspace, size_t workspace_bytes,
                     void* stream);

/*
 * The same aggregation for a caller whose gradients sit in HOST memory (ideally page-locked):
 * coordinate slabs are copied to the device workspace, aggregated there and the result is copied
 * back; the call returns after out_host is complete.  replicas_host is contiguous [r][f][d],
 * out_host is [d].  workspace: device, at least bz_workspace_bytes(BZ_OP_VOTE_MEDIAN_HOST, ...)
 * (more lets it use larger slabs, up to the whole array).
 */
int bz_vote_median_host(const float* replicas_host, int r, int f, int64_t d, float* out_host, void* workspace,
                        size_t workspace_bytes, void* stream);

/*
 * Squared Euclidean distances between all pairs of voted gradients, the O(f^2 d) part of the
 * Krum family (Sec. 1.2; cost in Appendix A.1): dist[a][b] = sum_j (v_a[j] - v_b[j])^2.
 * Three kernels compute it; results are reproducible from run to run with each.
 *   - Tensor cores (f = 25 or 49, d >= 8192, 16-byte aligned rows, ld a multiple of 4): every row
 *     is converted to 31-bit fixed point on a power-of-two scale of its own, the Gram matrix of
 *     the integers is formed exactly by 8-bit integer MMAs, and dist = |a|^2 + |b|^2 - 2ab is taken
 *     in binary64.  The only error is the rounding of a value to a multiple of its row's step
 *     2^(E-30), with 2^E one bit above the magnitudes the row showed first.  Rare larger values
 *     (the tail of a heavy-tailed gradient) are taken out of the contraction and added exactly in
 *     binary64; a row that keeps producing them gets a coarser step.  The kernel counts the
 *     values it rounded and bounds, for every pair and for EVERY input - also one whose rounding
 *     errors an attacker lined up - what the roundings can have done to the distance
 *     (Cauchy-Schwarz).  Where the bound exceeds 1e-7 relative, or a row holds infinities, NaNs
 *     or magnitudes beyond 2^60, the binary64 kernel below recomputes (decided on the device; the
 *     call stays asynchronous).  On gradients like the benchmark's the bound is ~3e-8 and the actual
 *     error ~1e-11.  Two rows closer than binary64 sums of their squared norms can resolve are
 *     reported at distance 0 if the bound on their true distance is below 1e-7 of the smallest
 *     non-zero distance either has; otherwise the binary64 kernel answers.
 *   - Binary64 difference form (f = 25 or 49; any d, rows on any 4-byte boundary): differences,
 *     squares and sums in double precision, the oracle's result to ~1e-15 whatever the data; about
 *     2.5x the time of the binary32 kernel.  It runs behind the first kernel, reads that kernel's
 *     flag and returns at once unless asked; and it answers alone for rows shorter than 8192 and
 *     for rows the first kernel cannot take (not 16-byte aligned, ld not a multiple of 4 - e.g.
 *     contiguous rows of a length that is not a multiple of 4: pad them and the first kernel runs,
 *     about twice as fast).
 *   - Binary32 difference form (every other shape, and bz_pairdist_static): differences and squares
 *     in binary32, added in binary32 inside blocks of at most 1024 coordinates (interleaved partial
 *     sums of at most 128 terms) and in binary64 across blocks, in a fixed order.  Its rounding
 *     errors are those of binary32 products and short binary32 sums: ~3e-9 relative on gradients,
 *     up to ~2e-6 on rows of a few hundred coordinates, with no bound of the first kernel's kind.
 * Environment: BZ_PAIRDIST_PATH=fp32 / =fp64 keeps every call on that kernel (fp64: where it
 * exists); =i8 takes the first kernel's result whatever its bound says (for testing it); read at
 * every call.
 * With =i8 the binary64 kernel still answers for rows the fixed point cannot hold and after a
 * kernel that stopped early (below).
 * The tensor-core kernel bounds every wait.  If one runs out the kernel stops early, says so in
 * the workspace, and the binary64 kernel recomputes the whole matrix on the same stream: the result
 * is complete either way, bz_pairdist_status() reports what happened and bz_pipeline_timeouts()
 * counts it.
 *   dist  device, double [f][f], symmetric with a zero diagonal; identical rows give exactly 0.
 *   workspace  device, bz_workspace_bytes(BZ_OP_PAIRDIST, 0, f, d, 0, 0) bytes, 256-byte aligned.
 */
int bz_pairdist(const float* voted, int f, int64_t d, int64_t ld, double* dist, void* workspace,
                size_t workspace_bytes, void* stream);

/*
 * What the distance stage of the last call that used `workspace` did (bz_pairdist, bz_multikrum,
 * bz_bulyan, bz_vote_pairdist, bz_vote_multikrum, bz_vote_bulyan with the same f).  Synchronises
 * `stream`, then writes a combination of the bits below to *status (host):
 *   BZ_STATUS_RECOMPUTED     the binary64 kernel's distances were returned although the tensor-core
 *                            kernel ran (its error bound, values without a fixed-point scale,
 *                            or an early stop asked for it)
 *   BZ_STATUS_STOPPED_EARLY  a bounded wait of the tensor-core kernel ran out; its distances were
 *                            recomputed and, in the calls that vote first, the voted rows were
 *                            rebuilt by the vote kernel.  Outputs are complete and correct, the
 *                            call was slow; a device that does this is not healthy.
 * 0 when the tensor-core kernel's result stands or that kernel did not run.
 */
#define BZ_STATUS_RECOMPUTED 1
#define BZ_STATUS_STOPPED_EARLY 2
int bz_pairdist_status(const void* workspace, int f, int32_t* status, void* stream);

/*
 * bz_pairdist for callers that have no device workspace to offer and may not allocate one.
 * (The paper has no counterpart to this call; it exists for the library's users.)  Such callers
 * are, for instance, an operator embedded in a framework that fixes its memory plan before the
 * run, a serving or training loop that cannot afford the device-wide synchronisation an
 * allocation may cause, or a tenant of a shared GPU held to a fixed memory budget.  They pass
 * inputs and outputs only; the partial sums go to an array of BZ_STATIC_SCRATCH_BYTES that is part
 * of the library image, so every GPU that loads the library holds those 4 MiB until the process
 * exits.  The call itself allocates and frees nothing.
 *   - Results are those of bz_pairdist's binary32 difference-form kernel (the only one this call
 *     uses; same summation order).
 *   - Shapes whose partial sums exceed the
 *     array are refused with BZ_ERR_STATIC_LIMIT before anything runs: f = 25 (0.9 MB) and f = 49
 *     (1.6 MB) fit, any other f fits up to 84; f from 85 to BZ_MAX_F is refused.
 *   - The first call on each device looks up the array's device address (the device must be
 *     current, as for every call).  Make that first call outside any stream capture.  The
 *     address is kept per device for the life of the process: after cudaDeviceReset() on a
 *     device this entry point must not be used on it again.
 *   - All calls share the one array and it keeps the previous call's contents.  The kernels
 *     overwrite or clear every element before reading it, so successive calls on one stream are
 *     independent; two calls that overlap on the GPU (different streams, several host threads)
 *     race on the array and must be serialised by the caller.
 *   voted device [f][d] with ld;  dist device double [f][f].
 */
#define BZ_STATIC_SCRATCH_BYTES (4u << 20)
int bz_pairdist_static(const float* voted, int f, int64_t d, int64_t ld, double* dist, void* stream);

/*
 * Multi-Krum selection on a distance matrix (Sec. 1.2: the gradient closest to its nearest
 * neighbours; Sec. 6.1 for the operand requirement f >= 2c+3).  score[a] = sum of the f-c-2
 * smallest dist[a][b], b != a, added in ascending order; rows are ranked by (score, index) and
 * the first m are written to selected (m = 1 is Krum).  c counts corrupted OPERANDS (files).
 *   dist device double [f][f];  selected device int32 [m].
 */
int bz_krum_select(const double* dist, int f, int c, int m, int32_t* selected, void* stream);

/*
 * Coordinate-wise mean of m selected rows: binary64 sum in the order of `selected`, divided by m,
 * rounded once to binary32.   selected device int32 [m], values in [0, f).
 */
int bz_mean_rows(const float* voted, int f, int64_t d, int64_t ld, const int32_t* selected, int m, float* out,
                 void* stream);

/*
 * Multi-Krum end to end: bz_pairdist, bz_krum_select, bz_mean_rows.
 *   out device [d];  selected device int32 [m];  dist device double [f][f] or NULL (then the
 *   matrix lives in the workspace);  workspace >= bz_workspace_bytes(BZ_OP_MULTIKRUM, 0, f, d, c, m).
 */
int bz_multikrum(const float* voted, int f, int64_t d, int64_t ld, int c, int m, float* out, int32_t* selected,
                 double* dist, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Bulyan, first stage (Sec. 1.2; requirement f >= 4c+3 from Sec. 6.1): theta = f - 2c rows are
 * picked one at a time.  With R the rows not yet picked, a pick takes the (score, index)-smallest
 * row of R, scores being Krum scores inside R with clamp(|R|-c-2, 1, |R|-1) neighbours.
 *   selected device int32 [f - 2c], in pick order.
 */
int bz_bulyan_select(const double* dist, int f, int c, int32_t* selected, void* stream);

/*
 * Bulyan, second stage - the trimmed mean around the median described in Sec. 1.2: per
 * coordinate, of the theta selected values the beta closest to their median (rank (theta-1)/2 in
 * total order) are averaged.  Closeness is |v - median| in binary32; the window grows from the
 * median outward, ties go to the lower side; the mean is a binary64 sum in ascending order
 * divided by beta, rounded once.   1 <= beta <= theta <= f.
 *   Any alignment works; rows and out that are 16-byte (8-byte) aligned, with ld a multiple of 4 (2),
 *   are read with 128-bit (64-bit) loads.
 */
int bz_trimmed_mean(const float* voted, int f, int64_t d, int64_t ld, const int32_t* selected, int theta,
                    int beta, float* out, void* stream);

/*
 * Bulyan end to end with theta = f - 2c, beta = theta - 2c.
 *   selected device int32 [f - 2c];  workspace >= bz_workspace_bytes(BZ_OP_BULYAN, 0, f, d, c, 0).
 */
int bz_bulyan(const float* voted, int f, int64_t d, int64_t ld, int c, float* out, int32_t* selected,
              void* workspace, size_t workspace_bytes, void* stream);

/*
 * bz_vote and bz_pairdist in one pass over the replicas: the winners of Eq. (3) are written to
 * `voted` and enter the distance sums of Sec. 1.2 from on-chip memory, so the voted rows are not
 * read back (4*f of the 4*(r*f + 2*f) bytes per coordinate the two calls move are saved).
 * voted is bit-identical to bz_vote's; dist is computed as in bz_pairdist (f = 25, 49 with r = 3, 5
 * and 7 x 49: the vote runs in front of the tensor-core kernel, with the same bound and fall-back;
 * BZ_PAIRDIST_PATH=fp32 puts it in front of the binary32 kernel instead).  Shapes without a fused
 * kernel (r*f outside {3,5}x{25,49} and 7x49, unaligned or short arrays) run the two calls.
 * Should a bounded wait of the single-pass kernel run out, `voted` and `dist` are incomplete when
 * that kernel ends; the call has already enqueued the repair behind it (bz_vote's kernel, then the
 * binary64 distances; both return at once when there is nothing to repair), so outputs are
 * complete once the stream is synchronised.  bz_pairdist_status() and bz_pipeline_timeouts() tell.
 * The same holds for bz_vote_multikrum and bz_vote_bulyan, which start with this call.
 *   replicas, ld_file, ld_replica as bz_vote;  voted device [f][d] with ld_voted (written);
 *   dist device double [f][f];  workspace as bz_pairdist.
 */
int bz_vote_pairdist(const float* replicas, int r, int f, int64_t d, int64_t ld_file, int64_t ld_replica, float* voted,
                     int64_t ld_voted, double* dist, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Multi-Krum from the replicas: bz_vote_pairdist, bz_krum_select, bz_mean_rows.  Arguments as
 * bz_multikrum, plus the replicas and the voted rows (written).
 */
int bz_vote_multikrum(const float* replicas, int r, int f, int64_t d, int64_t ld_file, int64_t ld_replica, int c, int m,
                      float* voted, int64_t ld_voted, float* out, int32_t* selected, double* dist, void* workspace,
                      size_t workspace_bytes, void* stream);

/* Bulyan from the replicas: bz_vote_pairdist, bz_bulyan_select, bz_trimmed_mean.  Arguments as bz_bulyan. */
int bz_vote_bulyan(const float* replicas, int r, int f, int64_t d, int64_t ld_file, int64_t ld_replica, int c,
                   float* voted, int64_t ld_voted, float* out, int32_t* selected, void* workspace,
                   size_t workspace_bytes, void* stream);

/*
 * Worst-case number of distorted files (Sec. 5.3.2 "exhaustive simulations"; Sec. 6.1: the
 * attacked set is the maximiser): over all q-subsets S of the K workers, the largest number of
 * files with at least r' = (r+1)/2 holders in S, and the lexicographically first S attaining it.
 *   worker_mask host uint64 [K] (bit x = holds file x), f <= 64, r <= 7, 0 <= q <= K <= 64.
 *   max_subsets: BZ_ERR_BUDGET if C(K, q) is larger (0 = no limit).
 *   c_max host int32 [1];  argmax host int32 [q] ascending (may be NULL);  n_subsets host (may be NULL).
 *   workspace device, bz_workspace_bytes(BZ_OP_WORST_CASE, ...) bytes.  Synchronises `stream`.
 */
int bz_worst_case(const uint64_t* worker_mask, int K, int f, int r, int q, uint64_t max_subsets, int32_t* c_max,
                  int32_t* argmax, uint64_t* n_subsets, void* workspace, size_t workspace_bytes, void* stream);

/*
 * One share of the same search, for several GPUs (or several calls): the q-subsets are dealt to `parts`
 * shares in fixed-size runs of the enumeration, share `part` (0 <= part < parts) evaluates its own, and the
 * maximum over all shares - by c_max, then by the lexicographically first argmax - is bz_worst_case's
 * result (Sec. 5.3.2; nothing else is exchanged).  A share that receives no run reports c_max = -1
 * (and leaves argmax alone).  n_subsets is C(K, q), the size of the whole search, for every share.
 * Arguments, limits and errors as bz_worst_case; BZ_ERR_INVALID_ARG for a part outside [0, parts).
 */
int bz_worst_case_part(const uint64_t* worker_mask, int K, int f, int r, int q, int part, int parts, uint64_t max_subsets,
                       int32_t* c_max, int32_t* argmax, uint64_t* n_subsets, void* workspace, size_t workspace_bytes,
                       void* stream);

/*
 * The same search for the placement bz_assign_mols(l, r) makes (Algorithm 2; Ramanujan Case 2 when
 * r == l), shortened by the design's symmetry: shifting all files by (i, j) -> (i + a, j + b) maps
 * worker (k, s) to (k, s + alpha_k*a + b), so the l*l translations permute the workers inside each
 * parallel class and leave the number of distorted files unchanged.  One set of workers per orbit
 * is evaluated - the smallest of the orbit in lexicographic order - which keeps both results of
 * bz_worst_case: c_max, and the lexicographically first maximiser.  The work drops by nearly l*l,
 * which moves the wall Sec. 6.1 reports for the exhaustive search (K = 49 and large q).
 *   l prime, l <= 7;  r odd, 3 <= r <= l;  0 <= q <= r*l.
 *   max_subsets: BZ_ERR_BUDGET if the number of orbits is larger (0 = no limit).
 *   c_max host int32 [1];  argmax host int32 [q] ascending (may be NULL);
 *   n_orbits host: sets evaluated = orbits of q-subsets under the translations (may be NULL).
 *   workspace device, bz_workspace_bytes(BZ_OP_WORST_CASE_MOLS, r, l*l, 0, 0, 0) bytes.
 * Synchronises `stream`.
 */
int bz_worst_case_mols(int l, int r, int q, uint64_t max_subsets, int32_t* c_max, int32_t* argmax,
                       uint64_t* n_orbits, void* workspace, size_t workspace_bytes, void* stream);

/*
 * One share of bz_worst_case_mols, as bz_worst_case_part is one of bz_worst_case: share `part` of `parts`
 * evaluates every parts-th run of the orbit enumeration; the maximum over the shares (by c_max, then by the
 * lexicographically first argmax) is the one-call result; an empty share reports c_max = -1.
 */
int bz_worst_case_mols_part(int l, int r, int q, int part, int parts, uint64_t max_subsets, int32_t* c_max, int32_t* argmax,
                            uint64_t* n_orbits, void* workspace, size_t workspace_bytes, void* stream);

/* The number of sets bz_worst_case_mols(l, r, q) evaluates.  Host only; needs no GPU. */
int bz_mols_orbit_count(int l, int r, int q, uint64_t* n_orbits);

/* Bytes of device workspace `op` needs for the given shape (arguments an op ignores may be 0). */
size_t bz_workspace_bytes(int op, int r, int f, int64_t d, int c, int m);

/* Static description of a status code; never NULL. */
const char* bz_status_string(int status);

/* Message of the last CUDA runtime error seen by the calling thread ("" if none). */
const char* bz_last_cuda_error(void);

/*
 * The TMA-staged kernels bound every wait on a shared-memory barrier; a wait that runs out makes
 * the kernel stop early and bump a device-side counter instead of hanging.  This reads that
 * counter (synchronously; 0 after any number of healthy launches) into *count (host).
 */
int bz_pipeline_timeouts(unsigned int* count);

/*
 * Measurement aid (no counterpart in the paper): reads `bytes` bytes of device memory once and
 * leaves the XOR of all its 64-bit words in *checksum (device).  staged == 0: 128-bit streaming
 * loads into registers; staged != 0: 32 KB chunks brought into shared memory by the bulk-copy
 * engine, four in flight per SM, the way the staged aggregation kernels read.  Timed on a buffer
 * much larger than the L2 it gives the read-only bandwidth of this GPU, the second denominator
 * (beside a copy) for the aggregation kernels, which read r*f words per word they write.
 *   buf device, 16-byte aligned; bytes a multiple of 8;  checksum device uint64 [1].
 */
int bz_stream_probe(const void* buf, size_t bytes, int staged, uint64_t* checksum, void* stream);

/*
 * Testing aid for the recovery described at bz_pairdist: while `on` is not 0, the loader threads of
 * the tensor-core distance kernels (given rows and vote in front) issue no loads, so that every
 * CTA's first bounded wait runs out after about a second and the call takes its repair path.
 * Nothing faults or hangs.  Off when the library is loaded; a per-device switch (the current
 * device's is set); not for production use.  Synchronous.
 */
int bz_debug_stall_pipeline(int on);

/*
 * Which kernel family the calling thread's last call dispatched to (vote, median, fused pass,
 * distances and the calls built on them); for tests and tuning, results never depend on it.
 *   BZ_PATH_STAGED      vote / median kernels fed by the TMA unit through shared memory
 *   BZ_PATH_REGISTERS   the same arithmetic with loads straight into registers (any alignment)
 *   BZ_PATH_GENERIC     run-time (r, f) kernels for shapes without a specialisation
 *   BZ_PATH_TENSOR      integer distances on the tensor cores (the binary64 kernel queued behind them)
 *   BZ_PATH_FP32        binary32 difference-form distances
 *   BZ_PATH_FP32_FUSED  vote and binary32 distances in one pass
 *   BZ_PATH_FP64        binary64 difference-form distances
 */
#define BZ_PATH_NONE 0
#define BZ_PATH_STAGED 1
#define BZ_PATH_REGISTERS 2
#define BZ_PATH_GENERIC 3
#define BZ_PATH_TENSOR 4
#define BZ_PATH_FP32 5
#define BZ_PATH_FP32_FUSED 6
#define BZ_PATH_FP64 7
int bz_last_path(void);

/* Number of kernels this library has launched from the calling process since it was loaded. */
uint64_t bz_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* BZ_H_ */
