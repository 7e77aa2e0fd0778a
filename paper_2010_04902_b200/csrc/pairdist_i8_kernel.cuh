// Pairwise squared distances of the Krum family (Sec. 1.2; cost in Appendix A.1) on the tensor cores,
// in exact integer arithmetic.
//
// The f x f matrix of squared distances is a contraction over the d coordinates, but in floating
// point only its difference form is accurate enough: gradients share a large per-coordinate mean, so
// |a|^2 + |b|^2 - 2ab cancels most of its digits.  Integers do not round.  Every value of row a is
// converted to 31-bit fixed point on the row's own power-of-two scale 2^(30 - E_a) (per CTA; it changes
// only when the row outgrows it), the fixed-point word is cut into four balanced signed bytes
//     q = s3*2^24 + s2*2^16 + s1*2^8 + s0,   -128 <= s_i <= 127,
// and the Gram matrix of the q's is the sum over slice pairs (i, j) of 2^(8(i+j)) S_i S_j^T.  Each
// S_i S_j^T is an 8-bit integer MMA (tcgen05, kind::i8) with 32-bit accumulators in tensor memory:
// exact, and independent of the order of the coordinates.  The slices are stacked along M and N, so
// one or two MMAs per 32 coordinates produce every block that is needed (a block whose transpose is
// not produced is counted twice).  The accumulators stay in tensor memory and are read back ("drained")
// every 512 tiles (32-bit headroom), when a row changes its scale and at the end; a drain combines the
// blocks in binary64 and adds
//     T[a][b] += 2^(E_a + E_b - 60) * sum_blocks weight * S_i S_j^T [a][b]
// to the CTA's partial matrix (in shared memory, written out once).  A finishing kernel forms, per CTA and
// then over CTAs in a fixed order,
//     D[a][b] = (T[a][a] + T[b][b]) - (T[a][b] + T[b][a]).
// Identical rows give identical integers and therefore exactly equal distances and D = 0.
//
// What is not exact is the conversion: a value of row a is rounded to a multiple of 2^(E_a - 30).  A CTA
// fixes E_a when it first meets the row: one bit above the power of two that bounds the magnitudes of
// its first step.  Values whose binary exponent lies within 7 of E_a keep all 24 bits; smaller ones are
// rounded, by at most half a step, and the converters count them (n_small: a superset, read off the top
// bytes).  With N_a^2 = sum of n_small * (step/2)^2 over CTAs (and over a row's successive scales) the
// computed distance obeys |D^ - D| <= 2 (N_a + N_b) sqrt(D^) + (N_a + N_b)^2 (Cauchy-Schwarz): a bound
// that holds for every input, also for rows whose rounding errors were arranged to line up.  The finishing
// kernel compares it with the library's distance tolerance and raises a flag when it does not fit; the
// caller then runs the binary64 difference-form kernel, which starts by looking at that flag.
// A later value that does not fit the row's scale (magnitude 2^E_a or more) is an outlier as long as the
// CTA has met at most kOutCap of them in that row - the rare large values of a heavy-tailed row: it
// enters the contraction as zero and its coordinate goes on a short list kept per CTA and row; the finishing
// kernel then adds, in binary64 and in a fixed order, what those coordinates really contribute to every
// pair.  Past kOutCap the row has outgrown its scale (gradients change magnitude from layer to layer):
// E_a is set anew from the current step, and the accumulators are read back first, because tensor memory
// holds integers on the old scale.  The other way round, rows that have left three bits or more of their
// scale unused for four steps get a finer one.
//
// Per 128-coordinate tile and SM: f*512 bytes from HBM (r times that with the vote in front),
// f*128 conversions, 4 or 8 MMA instructions.
//
// Every warp of a CTA sees every tile, so what a warp spends per tile on waiting, signalling and
// bookkeeping bounds the CTA's rate whatever the number of warps: the unit of work between two
// signals is therefore a step of TS tiles (up to 4, as many as shared memory holds), and a box holds all the
// rows (or, with copies, 13 to 25 of them).
//
// Roles in a CTA (one CTA per SM, tiles dealt round-robin): one thread issues TMA loads of boxes
// [R copies][FC rows][128 coordinates] into a ring of shared memory; W converter warps own fixed rows
// (row r belongs to warp r % W), vote them if there are copies, fix their scales and write the
// operand tiles (K-major, 128-byte swizzle) of a second ring; one thread issues the MMAs; four warps
// drain.  Every mbarrier wait is bounded; on expiry the CTA stops, marks its record (the host side then
// repairs the result with the binary64 kernel) and g_i8_timeouts is raised.  Loads are plain per-CTA loads.
// Every hand-off of shared memory between roles is an mbarrier arrival with release semantics paired with the
// waiter's acquire: converter -> loader (box read), converter -> MMA thread (operand tiles, exponents, flush
// request), MMA thread -> drain warps -> MMA thread.
#pragma once

#include <type_traits>

#include "umma.cuh"

namespace bz {

constexpr int kTK = 128;             // coordinates per tile = bytes per operand row
constexpr int kDrainWarps = 4;       // warps 0-3: one per 32 lanes of tensor memory
constexpr int kMmaWarp = 4;
constexpr int kTmaWarp = 5;
constexpr int kConvWarp0 = 6;
constexpr int kFlushTiles = 512;     // 2^9 tiles * 2^7 coordinates * 2^14 per product < 2^31
constexpr int kENone = -1000, kELo = -64, kEHi = 64;
constexpr int kCtlBytes = 3072;
// ints per CTA in the record the converters leave: the rows' exponents, their counts of values that may have
// been rounded, their counts of outliers, then the "bad" mark
// (kInfoN2: 64 doubles - the squared rounding budget a row used up under its earlier scales)
constexpr int kInfoE = 0, kInfoSmall = 64, kInfoOut = 128, kInfoN2 = 192, kInfoBad = 320, kInfoStride = 328;
// in CTA 0's record only: the ticket counter and the collected marks of the kernel that finishes the distances
constexpr int kInfoTicket = 321, kInfoMarks = 322;
constexpr int kLookEvery = 4;        // steps between two looks at whether rows would fit a finer scale
constexpr int kOutCap = 8;           // listed outliers per CTA and row; a row that has more gets a coarser scale
constexpr int kBadValues = 1;        // bits of the mark: a row holds values no fixed-point scale can carry
constexpr int kBadStopped = 2;       //                   a wait ran out and the CTA stopped early

__device__ unsigned int g_i8_timeouts = 0;
// Testing aid (bz_debug_stall_pipeline): while not 0 the loader threads issue nothing, so the first bounded
// wait of every CTA runs out and the launch ends the way it would after a lost load.
__device__ int g_i8_stall = 0;

// F rows, W converter warps, R copies per row (1: the rows are given), FC rows per box, NS boxes in the ring,
// TS tiles per step
template <int F, int W, int R, int FC, int NS, int TS> struct I8Shape {
    static constexpr int RP = F <= 32 ? 32 : 64;          // rows of one slice in an operand tile (f padded)
    static constexpr int SPM = 128 / RP;                   // slices stacked along M in one MMA
    static constexpr int NMMA = 4 / SPM;                   // MMAs per 32 coordinates
    static constexpr int kOpStageBytes = 4 * RP * kTK;     // one tile: slices 3, 2, 1, 0 one after the other
    static constexpr int kSlotBytes = TS * kOpStageBytes;  // a step = TS tiles
    static constexpr int kSlots = 2;
    static constexpr int kTmemCols = RP == 64 ? 512 : 128;
    static constexpr int kChunks = (F + FC - 1) / FC;      // boxes per tile (rows past f in the last one are filled with zeros by the TMA unit and skipped)
    static constexpr int RWC = (FC + W - 1) / W;           // rows of a box one converter warp may own
    static constexpr int kBoxFloats = R * FC * kTK;
    static constexpr int kBoxBytes = kBoxFloats * 4;
    static constexpr int kThreads = (kConvWarp0 + W) * 32;
    static constexpr int kPartialBytes = (F * F * 8 + 15) / 16 * 16;   // the CTA's partial matrix T
    static constexpr int kSmem = 1024 + kSlots * kSlotBytes + NS * kBoxBytes + kCtlBytes + kPartialBytes;
    static_assert(F <= 64, "at most 64 rows");
    static_assert(TS == 1 || TS == 2 || TS == 4, "step sizes that are tested");
    static_assert(kBoxBytes % 128 == 0, "TMA destinations are 128-byte aligned");
    static_assert(kSmem <= 227 * 1024, "shared memory");
    // MMA m covers slice indices m*SPM .. m*SPM+SPM-1 along M and m*SPM .. 3 along N
    static constexpr int mma_n(int m) { return (4 - m * SPM) * RP; }
    static constexpr int mma_col(int m) { return m == 0 ? 0 : 4 * RP; }
};

__device__ __forceinline__ int clamp_e(int e) { return e < kELo ? kELo : (e > kEHi ? kEHi : e); }

// weight of block (si, sj) (slice indices: slice value 3 - index) in T: 2^(8(6-si-sj)), doubled when
// the transposed block (sj, si) is not among the computed ones
template <int SPM> __device__ __forceinline__ double block_weight(int si, int sj) {
    const int twice = ((sj / SPM) * SPM <= si) ? 0 : 1;
    return __longlong_as_double(static_cast<long long>(1023 + 8 * (6 - si - sj) + twice) << 52);
}

// Four scaled coordinates of one row -> one 32-bit word per slice (byte k = coordinate k).
// q = round(t) (|q| <= 2^30); adding 128 to each of the three low bytes (carries ripple upward) and
// flipping their top bits afterwards leaves the balanced signed bytes.
__device__ __forceinline__ void slice4(const float4& t, uint32_t (&w)[4]) {
    const uint32_t x0 = static_cast<uint32_t>(__float2int_rn(t.x) + 0x00808080);
    const uint32_t x1 = static_cast<uint32_t>(__float2int_rn(t.y) + 0x00808080);
    const uint32_t x2 = static_cast<uint32_t>(__float2int_rn(t.z) + 0x00808080);
    const uint32_t x3 = static_cast<uint32_t>(__float2int_rn(t.w) + 0x00808080);
    // 4 x 4 byte transpose
    const uint32_t lo01 = __byte_perm(x0, x1, 0x5140), lo23 = __byte_perm(x2, x3, 0x5140);
    const uint32_t hi01 = __byte_perm(x0, x1, 0x7362), hi23 = __byte_perm(x2, x3, 0x7362);
    w[0] = __byte_perm(lo01, lo23, 0x5410) ^ 0x80808080u;
    w[1] = __byte_perm(lo01, lo23, 0x7632) ^ 0x80808080u;
    w[2] = __byte_perm(hi01, hi23, 0x5410) ^ 0x80808080u;
    w[3] = __byte_perm(hi01, hi23, 0x7632);
}

// the larger magnitude of a and b (any sign); a NaN in either comes through
__device__ __forceinline__ float max_abs_nan(float a, float b) {
    float m;
    asm("max.NaN.xorsign.abs.f32 %0, %1, %2;" : "=f"(m) : "f"(a), "f"(b));
    return m;
}

// the largest magnitude of a, b and c, one instruction
__device__ __forceinline__ float max_abs_nan3(float a, float b, float c) {
    float m;
    asm("max.NaN.abs.f32 %0, %1, %2, %3;" : "=f"(m) : "f"(a), "f"(b), "f"(c));
    return m;
}

// R = 1: distances of the rows of `map` ([f][d]).  R > 1: `map` covers replicas[r][f][d]; row i is the vote
// (Eq. 3, element by element on bit patterns) over its R copies, which is also written to
// voted[i*ld_voted + j] (16-byte aligned, ld_voted a multiple of 4).
template <int F, int W, int R, int FC, int NS, int TS>
__global__ void __launch_bounds__(I8Shape<F, W, R, FC, NS, TS>::kThreads, 1)
    pairdist_i8_kernel(const __grid_constant__ CUtensorMap map, int64_t d, float* __restrict__ voted, int64_t ld_voted,
                       double* __restrict__ tpart, int* __restrict__ info, int* __restrict__ olist) {
    using S = I8Shape<F, W, R, FC, NS, TS>;
    constexpr int RP = S::RP, SPM = S::SPM, NMMA = S::NMMA, NO = S::kSlots, CH = S::kChunks, RWC = S::RWC;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* op = base;
    float* in = reinterpret_cast<float*>(base + NO * S::kSlotBytes);
    unsigned char* ctl = base + NO * S::kSlotBytes + NS * S::kBoxBytes;
    double* tp_s = reinterpret_cast<double*>(ctl + kCtlBytes);
    uint64_t* op_full = reinterpret_cast<uint64_t*>(ctl);
    uint64_t* op_empty = op_full + NO;
    uint64_t* in_full = op_empty + NO;
    uint64_t* in_empty = in_full + NS;
    uint64_t* acc_ready = in_empty + NS;
    uint64_t* drain_go = acc_ready + 1;
    uint64_t* drained = drain_go + 1;
    volatile int* e_stage = reinterpret_cast<volatile int*>(drained + 1);  // [NO][64]: the rows' exponents as of a step
    volatile int* e_cur = e_stage + NO * 64;                                 // [64]: the rows' exponents now
    volatile int* op_flush = e_cur + 64;                                     // [NO]: some row's scale changes with this step
    volatile int* drain_stage = op_flush + NO;                               // which e_stage row a drain uses
    volatile int* drain_final = drain_stage + 1;                             // is it the last drain
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(const_cast<int*>(drain_final) + 1);
    volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* n_small = dead + 1;                                        // [64]: values of a row that may have been rounded
    volatile int* n_out = n_small + 64;                                      // [64]: outliers of a row
    // [64]: sum of count * (half a step)^2 over the row's earlier scales (8-byte aligned: padded to an even number of ints before it)
    volatile double* n2_done = reinterpret_cast<volatile double*>(n_out + 64 + (NO & 1));
    static_assert((2 * NO + 2 * NS + 3) * 8 + (NO * 64 + 64 + NO + 6 + 128) * 4 + 64 * 8 <= kCtlBytes, "control block");

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t n_tiles = (d + kTK - 1) / kTK;
    // tiles are dealt round-robin, so that at any moment the CTAs read neighbouring pieces of each row
    const int64_t my_tiles = (n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x;  // at least 1: the grid never exceeds n_tiles
    const int64_t my_steps = (my_tiles + TS - 1) / TS;                             // the last step may hold fewer tiles
    double* tp = tpart + static_cast<size_t>(blockIdx.x) * F * F;

    if (tid == 0) {
        for (int o = 0; o < NO; ++o) {
            mbar_init(&op_full[o], W);
            mbar_init(&op_empty[o], 1);
            op_flush[o] = 0;
        }
        for (int s = 0; s < NS; ++s) {
            mbar_init(&in_full[s], 1);
            mbar_init(&in_empty[s], W);
        }
        mbar_init(acc_ready, 1);
        mbar_init(drain_go, 1);
        mbar_init(drained, kDrainWarps);
        *dead = 0;
        info[blockIdx.x * kInfoStride + kInfoBad] = 0;
        if (blockIdx.x == 0) info[kInfoTicket] = info[kInfoMarks] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 64) {
        e_cur[tid] = kENone;
        n_small[tid] = 0;
        n_out[tid] = 0;
        n2_done[tid] = 0.0;
    }
    // rows f .. RP-1 of every slice stay zero for the whole run
    for (int e = tid; e < NO * S::kSlotBytes / 16; e += S::kThreads) reinterpret_cast<uint4*>(op)[e] = make_uint4(0, 0, 0, 0);
    for (int e = tid; e < F * F; e += S::kThreads) tp_s[e] = 0.0;
    fence_async_smem();
    if (warp == kMmaWarp) tmem_alloc(tmem_slot, S::kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp < kDrainWarps) {
        // ------------------------------------------------------------------ drain: tensor memory -> T
        const int L = warp * 32 + lane, g = L / RP, a = L % RP;
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);
        bool ok = true;
        for (uint32_t k = 0; ok; ++k) {
            // the first request may be a whole launch away: long naps, still bounded (about 10 s)
            if (!mbar_wait_live(drain_go, k & 1, dead, 20000) || !mbar_wait_live(acc_ready, k & 1, dead)) {
                ok = false;
                break;
            }
            tc_fence_after_sync();
            const volatile int* e_row = e_stage + *drain_stage * 64;
            const bool last = *drain_final != 0;
            const int e_a = a < F ? e_row[a] : 0;
            for (int ph = 0; ph < SPM; ++ph) {
                if (g == ph) {  // uniform over the warp
                    constexpr int NBLK = (NMMA == 1) ? 4 : 6;  // blocks a lane meets: 4 - m*SPM over the MMAs
                    for (int b0 = 0; b0 < F; b0 += 8) {
                        int32_t x[NBLK][8];
                        {
                            int q = 0;
#pragma unroll
                            for (int m = 0; m < NMMA; ++m)
#pragma unroll
                                for (int h = 0; h < 4 - m * SPM; ++h, ++q) tmem_ld8(lane_base + S::mma_col(m) + h * RP + b0, x[q]);
                        }
                        tmem_ld_wait();
                        double val[8];
#pragma unroll
                        for (int c = 0; c < 8; ++c) val[c] = 0.0;
                        {
                            int q = 0;
#pragma unroll
                            for (int m = 0; m < NMMA; ++m)
#pragma unroll
                                for (int h = 0; h < 4 - m * SPM; ++h, ++q) {
                                    const double w = block_weight<SPM>(m * SPM + g, m * SPM + h);
#pragma unroll
                                    for (int c = 0; c < 8; ++c) val[c] += w * static_cast<double>(x[q][c]);
                                }
                        }
                        if (a < F) {
#pragma unroll
                            for (int c = 0; c < 8; ++c)
                                if (b0 + c < F) {
                                    const double sc = __longlong_as_double(static_cast<long long>(1023 + e_a + e_row[b0 + c] - 60) << 52);
                                    tp_s[a * F + b0 + c] += val[c] * sc;
                                }
                        }
                    }
                }
                asm volatile("bar.sync 1, %0;" ::"n"(kDrainWarps * 32) : "memory");
            }
            if (last)  // the barrier above has ordered the last additions
                for (int e = tid; e < F * F; e += kDrainWarps * 32) tp[e] = tp_s[e];
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(drained);
            if (last) break;
        }
        if (!ok && lane == 0) atomicAdd(&g_i8_timeouts, 1u);
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------------ MMA issue
        if (lane == 0) {
            uint32_t n_flush = 0, have_acc = 0;
            int since = 0;
            bool ok = true;
            uint64_t desc0[NO];
#pragma unroll
            for (int o = 0; o < NO; ++o) desc0[o] = smem_desc_k128(smem_u32(op + static_cast<size_t>(o) * S::kSlotBytes));
            int o = 0;
            uint32_t phase = 0;
            // step my_steps carries no data: it hands over the final exponents for the last drain
            for (int64_t step = 0; step <= my_steps && ok; ++step) {
                if (!mbar_wait_live(&op_full[o], phase, dead)) {
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                const bool last = step == my_steps;
                // every converter has arrived, so nobody writes the flag until the slot is handed back
                const int wants = op_flush[o];
                if (wants) op_flush[o] = 0;
                if (have_acc && (wants || since > kFlushTiles - TS || last)) {
                    *drain_stage = o;
                    *drain_final = last ? 1 : 0;
                    mma_commit(acc_ready);
                    mbar_arrive(drain_go);
                    if (!mbar_wait_live(drained, n_flush & 1, dead)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    ++n_flush;
                    have_acc = 0;
                    since = 0;
                }
                if (last) break;
                uint64_t slot_desc = desc0[0];
#pragma unroll
                for (int k = 1; k < NO; ++k)
                    if (o == k) slot_desc = desc0[k];
                const int n_sub = static_cast<int>(my_tiles - TS * step < TS ? my_tiles - TS * step : TS);
                for (int sub = 0; sub < n_sub; ++sub) {
#pragma unroll
                    for (int ks = 0; ks < kTK / 32; ++ks) {
#pragma unroll
                        for (int m = 0; m < NMMA; ++m) {
                            // the start-address field counts 16-byte units and cannot carry out of its 14 bits
                            const uint64_t desc = slot_desc + static_cast<uint64_t>((sub * S::kOpStageBytes + m * SPM * RP * kTK + ks * 32) >> 4);
                            mma_s8(tmem_base + S::mma_col(m), desc, desc, idesc_s8(128, S::mma_n(m)), have_acc | (sub > 0) | (ks > 0));
                        }
                    }
                }
                mma_commit(&op_empty[o]);
                have_acc = 1;
                since += n_sub;
                if (++o == NO) {
                    o = 0;
                    phase ^= 1;
                }
            }
            if (!ok) atomicAdd(&g_i8_timeouts, 1u);
        }
    } else if (warp == kTmaWarp) {
        // ------------------------------------------------------------------ TMA producer
        // box order: step by step, box-row by box-row, first the earlier tile of the step then the later
        if (lane == 0) {
            bool ok = true;
            int s = 0, filled = 0;
            uint32_t phase = 0;
            int64_t issued = 0;
            const int64_t steps_to_load = *const_cast<volatile int*>(&g_i8_stall) ? 0 : my_steps;
            for (int64_t step = 0; step < steps_to_load && ok; ++step) {
                const int n_sub = static_cast<int>(my_tiles - TS * step < TS ? my_tiles - TS * step : TS);
                for (int c = 0; c < CH && ok; ++c) {
                    for (int sub = 0; sub < n_sub; ++sub) {
                        if (filled == NS) {
                            if (!mbar_wait_live(&in_empty[s], phase ^ 1, dead)) {
                                ok = false;
                                break;
                            }
                        } else {
                            ++filled;
                        }
                        const int64_t tile = blockIdx.x + (TS * step + sub) * gridDim.x;
                        mbar_expect_tx(&in_full[s], S::kBoxBytes);
                        tma_load_3d(in + static_cast<size_t>(s) * S::kBoxFloats, &map, &in_full[s], static_cast<int>(tile * kTK), c * FC, 0);
                        ++issued;
                        if (++s == NS) {
                            s = 0;
                            phase ^= 1;
                        }
                    }
                }
            }
            if (!ok) {
                atomicAdd(&g_i8_timeouts, 1u);
                // shared memory must outlive the loads already issued
                for (int64_t b = issued > NS ? issued - NS : 0; b < issued; ++b)
                    mbar_wait(&in_full[b % NS], static_cast<uint32_t>(b / NS) & 1);
            }
        }
    } else {
        // ------------------------------------------------------------------ converters: boxes -> operand tiles
        const int cw = warp - kConvWarp0;
        int unrepresentable = 0;
        bool ok = true;
        int s = 0, o = 0;
        uint32_t in_phase = 0, op_phase = 0;
        // this lane's place inside a row of a slice: 16-byte chunk lane/4 (swizzled with the row), word lane%4
        const uint32_t lane_word = (lane & 3) << 2;
        int tiles_left = static_cast<int>(my_tiles < (int64_t(1) << 30) ? my_tiles : (int64_t(1) << 30));
        // this lane's counts of possibly rounded values, one per row the warp owns (box-row cc, i-th row of it);
        // they meet in shared memory when a row changes its scale and at the end
        int small_acc[CH * RWC];
#pragma unroll
        for (int e = 0; e < CH * RWC; ++e) small_acc[e] = 0;
        // the largest scaled magnitude this lane has seen in each box-row since the last look
        float m_run[CH];
#pragma unroll
        for (int e = 0; e < CH; ++e) m_run[e] = 0.f;
        // what stays the same from step to step for each row the warp owns: its exponent (e_cur holds a copy for the
        // other roles) and this lane's byte offset inside a slice of the operand tile
        int e_reg[CH * RWC];
        uint32_t dst_off[CH * RWC];
#pragma unroll
        for (int cc = 0; cc < CH; ++cc) {
            const int off_cc = CH == 1 ? cw : ((cw - cc * FC) % W + W) % W;
#pragma unroll
            for (int i = 0; i < RWC; ++i) {
                const int r = cc * FC + off_cc + W * i;
                e_reg[cc * RWC + i] = kENone;
                // row r of a slice: 128 bytes per row, 16-byte chunk (lane/4) ^ (r%8) within it
                dst_off[cc * RWC + i] = static_cast<uint32_t>(r) * 128u + ((((lane >> 2) ^ (r & 7)) << 4) | lane_word);
            }
        }
        // One step.  FIRST: the CTA meets the rows for the first time and fixes their scales; kept apart from the
        // steps that follow so that their code carries none of it.
        auto convert_step = [&](auto first_tag, int64_t step) {
            constexpr bool FIRST = decltype(first_tag)::value;
            const int n_sub = tiles_left < TS ? tiles_left : TS;
            // this lane's coordinates in the first tile of the step (used by the vote's stores and the outlier lists)
            const int64_t j0 = (blockIdx.x + TS * step * gridDim.x) * kTK + 4 * lane;
            const uint32_t slot = smem_u32(op) + static_cast<uint32_t>(o) * S::kSlotBytes;
            bool raise = false, have_slot = false;
#pragma unroll 1
            for (int c = 0; c < CH && ok; ++c) {
                // rows of this box-row that belong to this warp: c*FC + off + W*i
                const int off = CH == 1 ? cw : ((cw - c * FC) % W + W) % W;
                float4 val[TS][RWC];
                int E[RWC];
#pragma unroll
                for (int sub = 0; sub < TS; ++sub) {
                    if (sub < n_sub) {
                        if (!mbar_wait_live(&in_full[s], in_phase, dead)) {
                            ok = false;
                            break;
                        }
                        const uint32_t src = smem_u32(in) + static_cast<uint32_t>(s) * S::kBoxBytes + 16 * lane;
                        const int64_t j = j0 + sub * static_cast<int64_t>(gridDim.x) * kTK;
#pragma unroll
                        for (int i = 0; i < RWC; ++i) {
                            const int fi = off + W * i;
                            if (fi < FC && c * FC + fi < F) {
                                uint4 w;
                                if constexpr (R == 1) {
                                    w = lds128(src + fi * (kTK * 4));
                                } else {
                                    uint4 x[R];
#pragma unroll
                                    for (int k = 0; k < R; ++k) x[k] = lds128(src + (k * FC + fi) * (kTK * 4));
                                    uint32_t cp[R];
#pragma unroll
                                    for (int k = 0; k < R; ++k) cp[k] = x[k].x;
                                    w.x = vote_bits<R>(cp);
#pragma unroll
                                    for (int k = 0; k < R; ++k) cp[k] = x[k].y;
                                    w.y = vote_bits<R>(cp);
#pragma unroll
                                    for (int k = 0; k < R; ++k) cp[k] = x[k].z;
                                    w.z = vote_bits<R>(cp);
#pragma unroll
                                    for (int k = 0; k < R; ++k) cp[k] = x[k].w;
                                    w.w = vote_bits<R>(cp);
                                }
                                val[sub][i] = make_float4(__uint_as_float(w.x), __uint_as_float(w.y), __uint_as_float(w.z), __uint_as_float(w.w));
                            }
                        }
                        // The box is in registers: hand it back.  The arrival is a release (the loads above are
                        // ordered before the producer's next write into the box), so it comes BEFORE this tile's
                        // global stores: a release waits for the stores its thread has in flight, and stores
                        // issued after it have the whole conversion to drain before the step's next arrival.
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&in_empty[s]);
                        if constexpr (R > 1) {
#pragma unroll
                            for (int i = 0; i < RWC; ++i) {
                                const int fi = off + W * i;
                                if (fi < FC && c * FC + fi < F) {
                                    const float4 w = val[sub][i];
                                    float* q = voted + (c * FC + fi) * ld_voted + j;
                                    if (j + 3 < d) {
                                        __stcs(reinterpret_cast<float4*>(q), w);
                                    } else {  // ragged end
                                        if (j < d) q[0] = w.x;
                                        if (j + 1 < d) q[1] = w.y;
                                        if (j + 2 < d) q[2] = w.z;
                                    }
                                }
                            }
                        }
                        if (++s == NS) {
                            s = 0;
                            in_phase ^= 1;
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < RWC; ++i) val[sub][i] = make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
                if (!ok) break;
                // Scale with the rows' exponents and look at the largest result: below 2^30 (and no NaN) the
                // rows convert as they are - nearly always.  Otherwise either the row is new to this CTA (its
                // exponent is fixed now, from the exact maximum of this step) or some values do not fit its
                // scale (they are listed and enter as zero).  All tiles of a step take the same exponents.
                int old[RWC];
#pragma unroll
                for (int i = 0; i < RWC; ++i)
                {
                    old[i] = kENone;
#pragma unroll
                    for (int cc = 0; cc < CH; ++cc)
                        if (cc == c) old[i] = e_reg[cc * RWC + i];
                }
                // Every kLookEvery-th step: did the warp's rows of this box-row leave three bits or more of their
                // scales unused ever since the last look?  Then they get finer ones (a row's magnitude falls as well
                // as rises from layer to layer, and a step that stays coarse costs precision for all the values that
                // follow).  As with every change of scale, the accumulators are read back before this step's
                // products are added.
                if (!FIRST && (step & (kLookEvery - 1)) == kLookEvery - 1) {
                    float seen = 0.f;
#pragma unroll
                    for (int cc = 0; cc < CH; ++cc) {
                        if (cc == c) {
                            seen = m_run[cc];
                            m_run[cc] = 0.f;
                        }
                    }
                    const uint32_t top = __reduce_max_sync(0xffffffffu, __float_as_uint(seen) & 0x7fffffffu);
                    const int finer = 28 - (static_cast<int>(top >> 23) - 127);  // the largest scaled value stays below 2^29
                    if (top != 0 && finer >= 3 && finer < 64) {
#pragma unroll
                        for (int i = 0; i < RWC; ++i) {
                            if (off + W * i < FC && c * FC + off + W * i < F && old[i] - finer >= kELo) {
                                const int row = c * FC + off + W * i;
                                int so_far = 0;
#pragma unroll
                                for (int cc = 0; cc < CH; ++cc) {
                                    if (cc == c) {
                                        so_far = small_acc[cc * RWC + i];
                                        small_acc[cc * RWC + i] = 0;
                                    }
                                }
                                so_far = __reduce_add_sync(0xffffffffu, so_far);
                                if (lane == 0) {
                                    const double half_step = __longlong_as_double(static_cast<long long>(1023 + old[i] - 31) << 52);
                                    n2_done[row] += static_cast<double>(so_far) * half_step * half_step;
                                    e_cur[row] = old[i] - finer;
                                }
#pragma unroll
                                for (int cc = 0; cc < CH; ++cc)
                                    if (cc == c) e_reg[cc * RWC + i] = old[i] - finer;
                                raise = true;
                            }
                        }
                        __syncwarp();
                    }
                }
                float4 t[TS][RWC];
                float m = 0.f;
                if constexpr (!FIRST) {
#pragma unroll
                    for (int i = 0; i < RWC; ++i) {
                        if (off + W * i < FC && c * FC + off + W * i < F) {
                            E[i] = kENone;
#pragma unroll
                            for (int cc = 0; cc < CH; ++cc)
                                if (cc == c) E[i] = e_reg[cc * RWC + i];
                            const float scale = __int_as_float((30 - E[i] + 127) << 23);
#pragma unroll
                            for (int sub = 0; sub < TS; ++sub) {
                                t[sub][i] = make_float4(val[sub][i].x * scale, val[sub][i].y * scale, val[sub][i].z * scale, val[sub][i].w * scale);
                                m = max_abs_nan3(max_abs_nan3(m, t[sub][i].x, t[sub][i].y), t[sub][i].z, t[sub][i].w);
                            }
                        }
                    }
                }
                if constexpr (!FIRST) {
#pragma unroll
                    for (int cc = 0; cc < CH; ++cc)
                        if (cc == c) m_run[cc] = max_abs_nan(m_run[cc], m);
                }
                if (FIRST || __any_sync(0xffffffffu, !(fabsf(m) < 1073741824.0f))) {
#pragma unroll
                    for (int i = 0; i < RWC; ++i) {
                        if (off + W * i < FC && c * FC + off + W * i < F) {
                            const int row = c * FC + off + W * i;
                            uint32_t m8 = 0;
#pragma unroll
                            for (int sub = 0; sub < TS; ++sub)
                                m8 = max(m8, max(max(__float_as_uint(val[sub][i].x) & 0x7fffffffu, __float_as_uint(val[sub][i].y) & 0x7fffffffu),
                                                 max(__float_as_uint(val[sub][i].z) & 0x7fffffffu, __float_as_uint(val[sub][i].w) & 0x7fffffffu)));
                            const int need = static_cast<int>(__reduce_max_sync(0xffffffffu, m8) >> 23) - 126;  // |v| < 2^need
                            if (need > 60) unrepresentable = 1;  // infinities, NaNs, magnitudes beyond 2^60
                            if constexpr (FIRST) {
                                // The row's first scale.  One or two values that stand three bits or more above all
                                // the others are outliers already (listed, fed as zero), up to four times over: a scale
                                // set by them would be coarse for everything that follows.
                                int fit = need, cnt = 0;
                                if (need <= 60) {
                                    for (int round = 0; round < 5; ++round) {  // the last round only measures what is left
                                        uint32_t top = 0;
#pragma unroll
                                        for (int sub = 0; sub < TS; ++sub) {
                                            const float* v4 = reinterpret_cast<const float*>(&val[sub][i]);
#pragma unroll
                                            for (int k = 0; k < 4; ++k) top = max(top, __float_as_uint(v4[k]) & 0x7fffffffu);
                                        }
                                        top = __reduce_max_sync(0xffffffffu, top);
                                        if (top == 0) {
                                            fit = kELo;  // nothing but zeros (left): the finest scale will do
                                            break;
                                        }
                                        fit = static_cast<int>(top >> 23) - 126;
                                        if (round == 4 || fit <= kELo + 8) break;
                                        const uint32_t high = static_cast<uint32_t>(fit - 3 + 126) << 23;  // 2^(fit - 3) and up
                                        int n_high = 0;
#pragma unroll
                                        for (int sub = 0; sub < TS; ++sub) {
                                            const float* v4 = reinterpret_cast<const float*>(&val[sub][i]);
#pragma unroll
                                            for (int k = 0; k < 4; ++k) n_high += (__float_as_uint(v4[k]) & 0x7fffffffu) >= high;
                                        }
                                        n_high = __reduce_add_sync(0xffffffffu, n_high);
                                        if (n_high > 2 || cnt + n_high > kOutCap) break;
#pragma unroll
                                        for (int sub = 0; sub < TS; ++sub) {
                                            float* v4 = reinterpret_cast<float*>(&val[sub][i]);
#pragma unroll
                                            for (int k = 0; k < 4; ++k) {
                                                const bool big = (__float_as_uint(v4[k]) & 0x7fffffffu) >= high;
                                                const unsigned mask = __ballot_sync(0xffffffffu, big);
                                                if (big) {
                                                    olist[(static_cast<size_t>(blockIdx.x) * 64 + row) * kOutCap + cnt + __popc(mask & ((1u << lane) - 1u))] =
                                                        static_cast<int>(j0 + sub * static_cast<int64_t>(gridDim.x) * kTK + k);
                                                    v4[k] = 0.f;
                                                }
                                                cnt += __popc(mask);
                                            }
                                        }
                                    }
                                    if (lane == 0 && cnt > 0) n_out[row] = cnt;
                                }
                                // one bit of headroom: the finer the step, the tighter the bound on the conversion error
                                E[i] = clamp_e(fit + 1);
                                if (lane == 0) e_cur[row] = E[i];
#pragma unroll
                                for (int cc = 0; cc < CH; ++cc)
                                    if (cc == c) e_reg[cc * RWC + i] = E[i];
                                const float scale = __int_as_float((30 - E[i] + 127) << 23);
#pragma unroll
                                for (int sub = 0; sub < TS; ++sub)
                                    t[sub][i] = make_float4(val[sub][i].x * scale, val[sub][i].y * scale, val[sub][i].z * scale, val[sub][i].w * scale);
                            } else if (need > E[i]) {  // (a constexpr-else: steps after the first)
                                // values of magnitude 2^E or more: how many?
                                int total = 0;
#pragma unroll
                                for (int sub = 0; sub < TS; ++sub) {
                                    if (sub < n_sub) {
                                        const float* tv = reinterpret_cast<const float*>(&t[sub][i]);
#pragma unroll
                                        for (int k = 0; k < 4; ++k) total += !(fabsf(tv[k]) < 1073741824.0f);
                                    }
                                }
                                total = __reduce_add_sync(0xffffffffu, total);
                                int cnt = n_out[row];
                                if (cnt + total <= kOutCap) {
                                    // few: outliers.  They enter as zero and are listed in the fixed order (tile, component, lane)
#pragma unroll
                                    for (int sub = 0; sub < TS; ++sub) {
                                        if (sub < n_sub) {
                                            float* tv = reinterpret_cast<float*>(&t[sub][i]);
#pragma unroll
                                            for (int k = 0; k < 4; ++k) {
                                                const bool big = !(fabsf(tv[k]) < 1073741824.0f);
                                                const unsigned mask = __ballot_sync(0xffffffffu, big);
                                                if (big) {
                                                    olist[(static_cast<size_t>(blockIdx.x) * 64 + row) * kOutCap + cnt + __popc(mask & ((1u << lane) - 1u))] =
                                                        static_cast<int>(j0 + sub * static_cast<int64_t>(gridDim.x) * kTK + k);
                                                    tv[k] = 0.f;
                                                }
                                                cnt += __popc(mask);
                                            }
                                        }
                                    }
                                    __syncwarp();
                                    if (lane == 0) n_out[row] = cnt;
                                } else {
                                    // many: the row has outgrown its scale (gradients change magnitude from layer to layer).
                                    // New exponent from this step's exact maximum; the accumulators are read back before
                                    // this step's products are added, and the roundings counted so far are charged at the
                                    // old step.
                                    int so_far = 0;
#pragma unroll
                                    for (int cc = 0; cc < CH; ++cc) {
                                        if (cc == c) {
                                            so_far = small_acc[cc * RWC + i];
                                            small_acc[cc * RWC + i] = 0;
                                        }
                                    }
                                    so_far = __reduce_add_sync(0xffffffffu, so_far);
                                    if (lane == 0) {
                                        const double half_step = __longlong_as_double(static_cast<long long>(1023 + E[i] - 31) << 52);
                                        n2_done[row] += static_cast<double>(so_far) * half_step * half_step;
                                    }
                                    raise = true;
                                    E[i] = clamp_e(need + 1);
                                    if (lane == 0) e_cur[row] = E[i];
#pragma unroll
                                    for (int cc = 0; cc < CH; ++cc)
                                        if (cc == c) e_reg[cc * RWC + i] = E[i];
                                    const float scale = __int_as_float((30 - E[i] + 127) << 23);
#pragma unroll
                                    for (int sub = 0; sub < TS; ++sub)
                                        t[sub][i] = make_float4(val[sub][i].x * scale, val[sub][i].y * scale, val[sub][i].z * scale, val[sub][i].w * scale);
                                    __syncwarp();
                                }
                            }
                        }
                    }
                }
                // the operand slot is free once the MMAs of step - NO are done
                if (!have_slot) {
                    if (step >= NO && !mbar_wait_live(&op_empty[o], op_phase ^ 1, dead)) {
                        ok = false;
                        break;
                    }
                    have_slot = true;
                }
#pragma unroll
                for (int i = 0; i < RWC; ++i) {
                    const int fi = off + W * i;
                    if (fi < FC && c * FC + fi < F) {
                        const int r = c * FC + fi;
                        // a row whose scale changes hands its old exponent to the drain that comes before this step
                        if (lane == 0) e_stage[o * 64 + r] = FIRST ? E[i] : old[i];
                        uint32_t my_off = 0;
#pragma unroll
                        for (int cc = 0; cc < CH; ++cc)
                            if (cc == c) my_off = dst_off[cc * RWC + i];
                        const uint32_t dst = slot + my_off;
                        int small = 0;
#pragma unroll
                        for (int sub = 0; sub < TS; ++sub) {
                            if (sub < n_sub) {
                                uint32_t w[4];
                                slice4(t[sub][i], w);
                                sts32(dst + sub * S::kOpStageBytes + 0 * RP * kTK, w[3]);
                                sts32(dst + sub * S::kOpStageBytes + 1 * RP * kTK, w[2]);
                                sts32(dst + sub * S::kOpStageBytes + 2 * RP * kTK, w[1]);
                                sts32(dst + sub * S::kOpStageBytes + 3 * RP * kTK, w[0]);
                                // A value can only have been rounded if |q| <= 2^23, and then its top byte (of
                                // q + 0x808080) is 0 or 1: count the bytes of that word whose upper seven bits are
                                // clear (a zero-byte test; the bytes tested are even, so it has no false positives).
                                const uint32_t z = w[3] & 0xfefefefeu;
                                small += __popc((z - 0x01010101u) & ~z & 0x80808080u);
                            }
                        }
#pragma unroll
                        for (int cc = 0; cc < CH; ++cc)
                            if (cc == c) small_acc[cc * RWC + i] += small;
                    }
                }
            }
            if (!ok) return;
            if (!have_slot && step >= NO && !mbar_wait_live(&op_empty[o], op_phase ^ 1, dead)) {
                ok = false;
                return;
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
                if (raise) atomicOr(const_cast<int*>(&op_flush[o]), 1);
                // release: this warp's operand tiles, exponents and flush request are ordered before whatever
                // the MMA thread (and, through its own arrivals, the drain warps) does after its wait
                mbar_arrive(&op_full[o]);
            }
            if (++o == NO) {
                o = 0;
                op_phase ^= 1;
            }
        };
        if (my_steps > 0) {
            convert_step(std::true_type{}, 0);
            tiles_left -= TS;
        }
        for (int64_t step = 1; step < my_steps && ok; ++step, tiles_left -= TS) convert_step(std::false_type{}, step);
        if (ok) {
            // the slot after the last step: current exponents, nothing to multiply
            if (my_steps >= NO && !mbar_wait_live(&op_empty[o], op_phase ^ 1, dead)) ok = false;
            if (ok) {
                if (lane == 0)
                    for (int r = cw; r < F; r += W) e_stage[o * 64 + r] = e_cur[r];
                __syncwarp();
                if (lane == 0) mbar_arrive(&op_full[o]);
            }
        }
        if (!ok && lane == 0) atomicAdd(&g_i8_timeouts, 1u);
#pragma unroll
        for (int cc = 0; cc < CH; ++cc) {
            const int off = CH == 1 ? cw : ((cw - cc * FC) % W + W) % W;
#pragma unroll
            for (int i = 0; i < RWC; ++i) {
                const int total = __reduce_add_sync(0xffffffffu, small_acc[cc * RWC + i]);
                if (lane == 0 && off + W * i < FC && cc * FC + off + W * i < F) n_small[cc * FC + off + W * i] = total;
            }
        }
        __syncwarp();
        if (lane == 0) {
            for (int r = cw; r < F; r += W) {
                info[blockIdx.x * kInfoStride + kInfoE + r] = e_cur[r];
                info[blockIdx.x * kInfoStride + kInfoSmall + r] = n_small[r];
                info[blockIdx.x * kInfoStride + kInfoOut + r] = n_out[r];
                reinterpret_cast<double*>(info + blockIdx.x * kInfoStride + kInfoN2)[r] = n2_done[r];
            }
            if (unrepresentable) atomicOr(&info[blockIdx.x * kInfoStride + kInfoBad], kBadValues);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    // whichever role's wait ran out first has raised `dead`: the CTA's partial matrix (and, with the vote in
    // front, its share of the voted rows) is incomplete
    if (tid == 0 && *dead) atomicOr(&info[blockIdx.x * kInfoStride + kInfoBad], kBadStopped);
    if (warp == kMmaWarp) tmem_dealloc(tmem_base, S::kTmemCols);
}

}  // namespace bz
