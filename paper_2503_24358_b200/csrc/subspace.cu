// Step 1 of the write path: query subspace and update matrices, all in fp64.
//
//   gram_kernel      M_h = Qc^T Qc for the stacked prompt queries of KV head h (Section 3.2;
//                    Algorithm 1 line 5 needs only the right singular vectors and singular values
//                    of Qc, i.e. the eigen-pairs of M_h; GQA stacking rule of Appendix C).
//   eig_cluster_kernel  eigen-decomposition of M_h: Cholesky M_h + shift I = L L^T, then one-sided (Hestenes)
//                    Jacobi on the columns of L: rotations make the columns orthogonal, L V = U Sigma;
//                    the normalised columns U are the eigenvectors v_i of M_h and the squared column
//                    norms, minus the shift, its eigenvalues sigma_i^2.
//   assemble_kernel  P_inv = (I + lambda Qhat^T Qhat)^{-1} = I - sum_i s_i/(1+s_i) v_i v_i^T with
//                    s_i = lambda sigma_i^2 (Woodbury with orthonormal v_i; footnote of Prop. 4),
//                    then the update matrices B_t H_t of Lemma 3 read off the LDL^T factorisation
//                    P_inv = (I+W) D (I+W)^T: for g = 1, I+W is its unit lower factor (this equals
//                    the chain of Prop. 2 / Lemma 4 followed by B_t h_t, which the CPU oracle runs
//                    literally); for g > 1 each block column is multiplied by the inverse of its
//                    unit-lower diagonal block, which turns the scalar factor into the block one.
//
// The cut at rank r can fall between nearly equal eigenvalues whose directions still carry
// weight lambda sigma^2, so single precision anywhere in this step changes quantized codes
// downstream; products of bf16 inputs are exact in fp64 and everything stays fp64 until W is
// rounded to float32 at the very end.
#include <cooperative_groups.h>
#include "squat_internal.cuh"

namespace {

constexpr int D = SQUAT_D;

// ------------------------------------------------------------------------------------- Gram
constexpr int GRAM_THREADS = 160;   // 136 upper-triangular 8x8 tiles of the 16x16 tile grid, 5 warps
constexpr int GRAM_ROWS = 32;       // rows staged in shared memory per step

template <bool BF16>
__global__ void __launch_bounds__(GRAM_THREADS) gram_kernel(
    const void *__restrict__ q, int n_tokens, int q_per_kv, long long stride_h, long long stride_t,
    int rows_per_chunk, double *__restrict__ partial /* [chunks, H, D, D] */)
{
    __shared__ __align__(16) double rows[GRAM_ROWS][D];
    const int h = blockIdx.y, chunk = blockIdx.x, H = gridDim.y;
    const long long N = (long long)n_tokens * q_per_kv;
    const long long row_lo = (long long)chunk * rows_per_chunk;
    long long row_hi = row_lo + rows_per_chunk;
    if (row_hi > N) row_hi = N;

    // tile of this thread: (ti <= tj) in the 16 x 16 grid of 8 x 8 tiles
    int ti = 0, tj = 0;
    {
        int t = threadIdx.x, rowlen = 16;
        while (t >= rowlen && ti < 15) { t -= rowlen; --rowlen; ++ti; }
        tj = ti + t;
    }
    const bool active = threadIdx.x < 136;
    double acc[8][8];
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 8; ++b) acc[a][b] = 0.0;

    // Each thread stages up to 4 pieces of 8 elements per step (32 rows x 16 pieces over 160 threads).  The
    // global loads of step s+1 are issued before the arithmetic of step s, so their latency is hidden.
    constexpr int NPIECE = (GRAM_ROWS * (D / 8) + GRAM_THREADS - 1) / GRAM_THREADS;
    uint4 pre[NPIECE][BF16 ? 1 : 2];
    auto fetch = [&](long long r0) {
#pragma unroll
        for (int it = 0; it < NPIECE; ++it) {
            const int idx = threadIdx.x + it * GRAM_THREADS;
            const int rr = idx / (D / 8), c8 = idx % (D / 8);
            const long long n = r0 + rr;
            if (idx < GRAM_ROWS * (D / 8) && n < row_hi) {
                const long long hq = (long long)h * q_per_kv + n / n_tokens;
                const long long t = n % n_tokens;
                const long long off = hq * stride_h + t * stride_t + c8 * 8;
                if (BF16) {
                    pre[it][0] = ldg128(reinterpret_cast<const __nv_bfloat16 *>(q) + off);
                } else {
                    pre[it][0] = ldg128(reinterpret_cast<const float *>(q) + off);
                    pre[it][BF16 ? 0 : 1] = ldg128(reinterpret_cast<const float *>(q) + off + 4);
                }
            } else {
                pre[it][0] = make_uint4(0, 0, 0, 0);
                pre[it][BF16 ? 0 : 1] = make_uint4(0, 0, 0, 0);
            }
        }
    };
    if (row_lo < row_hi) fetch(row_lo);
    for (long long r0 = row_lo; r0 < row_hi; r0 += GRAM_ROWS) {
        __syncthreads();
#pragma unroll
        for (int it = 0; it < NPIECE; ++it) {
            const int idx = threadIdx.x + it * GRAM_THREADS;
            if (idx >= GRAM_ROWS * (D / 8)) continue;
            const int rr = idx / (D / 8), c8 = idx % (D / 8);
            double v[8];
            if (BF16) {
                const uint32_t w[4] = {pre[it][0].x, pre[it][0].y, pre[it][0].z, pre[it][0].w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    v[2 * k] = (double)bf16lo_to_f32(w[k]);
                    v[2 * k + 1] = (double)bf16hi_to_f32(w[k]);
                }
            } else {
                const uint4 a = pre[it][0], b = pre[it][BF16 ? 0 : 1];
                v[0] = __uint_as_float(a.x); v[1] = __uint_as_float(a.y); v[2] = __uint_as_float(a.z); v[3] = __uint_as_float(a.w);
                v[4] = __uint_as_float(b.x); v[5] = __uint_as_float(b.y); v[6] = __uint_as_float(b.z); v[7] = __uint_as_float(b.w);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) rows[rr][c8 * 8 + k] = v[k];
        }
        __syncthreads();
        if (r0 + GRAM_ROWS < row_hi) fetch(r0 + GRAM_ROWS);
        if (active) {
#pragma unroll 4
            for (int rr = 0; rr < GRAM_ROWS; ++rr) {
                double a[8], b[8];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const double2 va = *reinterpret_cast<const double2 *>(&rows[rr][ti * 8 + 2 * k]);
                    const double2 vb = *reinterpret_cast<const double2 *>(&rows[rr][tj * 8 + 2 * k]);
                    a[2 * k] = va.x; a[2 * k + 1] = va.y;
                    b[2 * k] = vb.x; b[2 * k + 1] = vb.y;
                }
#pragma unroll
                for (int x = 0; x < 8; ++x)
#pragma unroll
                    for (int y = 0; y < 8; ++y) acc[x][y] = fma(a[x], b[y], acc[x][y]);
            }
        }
    }
    if (active) {
        double *out = partial + ((long long)chunk * H + h) * D * D;
#pragma unroll
        for (int x = 0; x < 8; ++x)
#pragma unroll
            for (int y = 0; y < 8; ++y) out[(ti * 8 + x) * D + tj * 8 + y] = acc[x][y];
    }
}

// Sums the per-chunk partials in a fixed order and mirrors the upper tiles: gram[h] full symmetric.
__global__ void gram_reduce_kernel(const double *__restrict__ partial, int chunks, int H, double *__restrict__ gram)
{
    const int h = blockIdx.y;
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= D * D) return;
    int a = idx / D, b = idx % D;
    if (a / 8 > b / 8) { const int t = a; a = b; b = t; }       // read from the stored upper tile
    double s = 0.0;
    for (int c = 0; c < chunks; ++c) s += partial[((long long)c * H + h) * D * D + a * D + b];
    gram[(long long)h * D * D + idx] = s;
}

// ------------------------------------------------------------------------------------- eigen
constexpr int EIG_LD = D + 2;       // padded column stride (doubles) of the full matrix
constexpr int EIG_MAX_SWEEPS = 40;

// Eigen-decomposition of M: Cholesky M + shift I = L L^T, then one-sided (Hestenes) Jacobi on the columns of L
// (cyclic tournament order, 64 disjoint column pairs per round, cached squared norms, rotations skipped below
// 1e-14 relative).  L has the square root of M's condition number and L^T L is much closer to diagonal than
// M^2, which cuts the sweeps (14 -> 10 on the 4096-token workload).  The shift (1e-12 of the trace) keeps
// the factorisation defined for rank-deficient M and is subtracted from the eigenvalues at the end;
// eigenvectors are unaffected by it.  Jacobi converges quadratically, so a sweep in which every pair starts
// below 1e-7 relative leaves them below ~1e-14: that sweep is the last.
//
// The rows of L are split over a cluster of 4 CTAs (4 SMs per head instead of 1; a
// 32-head layer then occupies 128 of the 148 SMs).  Column rotations act on every row independently, so each
// CTA rotates its own 32-row slice; only the dot product of a column pair needs all rows: every CTA writes its
// partial sums into the shared memory of all four (distributed shared memory), one hardware cluster barrier
// per round, and then all four CTAs add the partials in the same order -- every CTA takes bit-identical
// rotation decisions, so they stay in step without further communication.  The Cholesky factorisation is
// done redundantly by each CTA on a full copy (it is a small part of the time).
namespace cg = cooperative_groups;
constexpr int ECL = 4;                       // CTAs per cluster
constexpr int ECT = 512;                     // threads per CTA: 64 column pairs x 8 lanes
constexpr int ESL_ROWS = D / ECL;            // rows per CTA (32)
constexpr int ESL_LD = ESL_ROWS + 2;         // padded column stride of the slice
constexpr int ESL_RPL = ESL_ROWS / 8;        // rows per lane (4)

__device__ __forceinline__ double team8_sum(double v)
{
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    v += __shfl_xor_sync(0xffffffffu, v, 2);
    v += __shfl_xor_sync(0xffffffffu, v, 4);
    return v;
}

__device__ __forceinline__ double team16_sum(double v)
{
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    v += __shfl_xor_sync(0xffffffffu, v, 2);
    v += __shfl_xor_sync(0xffffffffu, v, 4);
    v += __shfl_xor_sync(0xffffffffu, v, 8);
    return v;
}

// 1/sqrt(x) for a normal positive double: hardware seed y (relative error 2^-22), residual r = 1 - x y^2, and one
// third-order correction y (1 + r/2 + 3 r^2/8); what is left, about r^3/3, is far below a double's rounding.
__device__ __forceinline__ double rsqrt_nr(double x)
{
    double y;
    asm("rsqrt.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(x));
    const double r = fma(-(x * y), y, 1.0);
    return fma(y * r, fma(0.375, r, 0.5), y);
}

// One stage of the Jacobi method on the 4 x 4 Gram matrix g of a 4-column set: the two rotations (P,Q) and (R,S) act
// on disjoint planes, so both are decided from the current g and applied together, free of branches (the two
// dependency chains interleave).  A rotation turns col P into c colP - s colQ and col Q into s colP + c colQ with the
// angle that makes them orthogonal (tan 2theta = 2 g_PQ / (g_QQ - g_PP), |theta| <= pi/4), from two reciprocal
// square roots.  A pair already orthogonal to 1e-14 relative, or numerically null twice over, keeps c = 1, s = 0.
struct RotParams { double c, s, t; bool act; };

__device__ __forceinline__ RotParams rot_params(double alpha, double beta, double gam, double null_thr, double tol2, int &big)
{
    RotParams p;
    const double g2 = gam * gam, ab = alpha * beta;
    p.act = (alpha > null_thr || beta > null_thr) && g2 > tol2 * ab;
    const double diff = beta - alpha;
    const double rr = fma(diff, diff, 4.0 * g2);
    const double inv_r = rsqrt_nr(p.act ? rr : 1.0);
    const double hc = fma(0.5 * fabs(diff), inv_r, 0.5);              // (1 + cos 2theta)/2 = c^2, in [1/2, 1]
    const double inv_c = rsqrt_nr(p.act ? hc : 1.0);
    const double sm = gam * inv_r * inv_c;
    p.c = p.act ? hc * inv_c : 1.0;
    p.s = p.act ? (diff < 0.0 ? -sm : sm) : 0.0;
    p.t = p.s * inv_c;                                                // tan(theta)
    if (p.act && g2 > 1e-14 * ab) big = 1;
    return p;
}

template <int P, int Q, int R, int S>
__device__ __forceinline__ void gram_stage(double (&g)[4][4], double null_thr, double tol2,
                                           double &c1, double &s1, double &c2, double &s2, int &big)
{
    const RotParams a = rot_params(g[P][P], g[Q][Q], g[P][Q], null_thr, tol2, big);
    const RotParams b = rot_params(g[R][R], g[S][S], g[R][S], null_thr, tol2, big);
    const double gpq = g[P][Q], grs = g[R][S];
    g[P][P] -= a.t * gpq;
    g[Q][Q] += a.t * gpq;
    g[R][R] -= b.t * grs;
    g[S][S] += b.t * grs;
    g[P][Q] = g[Q][P] = a.act ? 0.0 : gpq;
    g[R][S] = g[S][R] = b.act ? 0.0 : grs;
    // the 2 x 2 block between the planes: rotate its (P,Q) index by a, then its (R,S) index by b
    const double pr = a.c * g[P][R] - a.s * g[Q][R], qr = a.s * g[P][R] + a.c * g[Q][R];
    const double ps = a.c * g[P][S] - a.s * g[Q][S], qs = a.s * g[P][S] + a.c * g[Q][S];
    g[P][R] = g[R][P] = b.c * pr - b.s * ps;
    g[P][S] = g[S][P] = b.s * pr + b.c * ps;
    g[Q][R] = g[R][Q] = b.c * qr - b.s * qs;
    g[Q][S] = g[S][Q] = b.s * qr + b.c * qs;
    c1 = a.c; s1 = a.s; c2 = b.c; s2 = b.s;
}

__global__ void __cluster_dims__(ECL, 1, 1) __launch_bounds__(ECT, 1) eig_cluster_kernel(
    const double *__restrict__ gram, double *__restrict__ eigval, double *__restrict__ eigvec,
    int *__restrict__ sweeps_out, unsigned *__restrict__ status)
{
    cg::cluster_group cluster = cg::this_cluster();
    const int crank = (int)cluster.block_rank();
    extern __shared__ __align__(16) double sm[];
    double *Gs = sm;                                   // full matrix for the factorisation: Gs[col * EIG_LD + row]
    double *Gl = Gs + D * EIG_LD;                      // this CTA's row slice: Gl[col * ESL_LD + r]
    double *gpart = Gl + D * ESL_LD;                   // [2 parities][ECL sources][10 entries][32 teams] partial Gram sums
    double *npart = gpart + 2 * ECL * 32 * 10;              // [ECL sources][D] partial squared norms
    double *nrm = npart + ECL * D;                     // [D] column norms (identical in every CTA)
    double *rotcs = nrm + D;                           // [32 teams][6 rotations] (c, s) of the current round
    int *rank = reinterpret_cast<int *>(rotcs + 32 * 12);
    const int h = blockIdx.x / ECL, tid = threadIdx.x;
    const int team = tid >> 3, l8 = tid & 7;
    const double *M = gram + (long long)h * D * D;

    for (int idx = tid; idx < D * D; idx += ECT) {
        const int r = idx / D, c = idx % D;
        Gs[c * EIG_LD + r] = M[idx];
    }
    __syncthreads();
    double trace = 0.0;
    for (int i = 0; i < D; ++i) trace += Gs[i * EIG_LD + i];
    const double shift = trace > 0.0 ? 1e-12 * trace : 1e-300;       // M + shift I = L L^T
    __syncthreads();
    if (tid < D) Gs[tid * EIG_LD + tid] += shift;
    double *lcol = nrm;
    for (int j = 0; j < D; ++j) {
        __syncthreads();
        const double ajj = Gs[j * EIG_LD + j];
        const double ljj = sqrt(ajj > 0.0 ? ajj : shift);
        if (tid >= j && tid < D) lcol[tid] = (tid == j) ? ljj : Gs[j * EIG_LD + tid] / ljj;
        __syncthreads();
        // trailing update of the lower triangle (row >= col); 2-D thread grid, no index division
        for (int c = j + 1 + (tid >> 5); c < D; c += ECT / 32) {
            const double lc = lcol[c];
            for (int r = c + (tid & 31); r < D; r += 32) Gs[c * EIG_LD + r] = fma(-lcol[r], lc, Gs[c * EIG_LD + r]);
        }
        if (tid >= j && tid < D) Gs[j * EIG_LD + tid] = lcol[tid];
    }
    __syncthreads();
    // keep rows [32 crank, 32 crank + 32) of L (lower triangular: zero above the diagonal)
    for (int idx = tid; idx < D * ESL_ROWS; idx += ECT) {
        const int c = idx / ESL_ROWS, r = idx % ESL_ROWS, gr = crank * ESL_ROWS + r;
        Gl[c * ESL_LD + r] = (gr >= c) ? Gs[c * EIG_LD + gr] : 0.0;
    }
    const double null_thr = 4.0 * shift;
    const double tol2 = 1e-14 * 1e-14;
    cluster.sync();                                    // every CTA's shared memory is set up before remote writes

    double *gpart_remote[ECL], *npart_remote[ECL];
#pragma unroll
    for (int r = 0; r < ECL; ++r) {
        gpart_remote[r] = cluster.map_shared_rank(gpart, r);
        npart_remote[r] = cluster.map_shared_rank(npart, r);
    }

    // squared norms of all columns: partial over the local rows, exchanged, summed in rank order
    auto refresh_norms = [&](bool take_sqrt) {
        for (int col = team; col < D; col += ECT / 8) {
            double s = 0.0;
#pragma unroll
            for (int i = 0; i < ESL_RPL; ++i) { const double v = Gl[col * ESL_LD + l8 + 8 * i]; s = fma(v, v, s); }
            s = team8_sum(s);
            if (l8 < ECL) npart_remote[l8][crank * D + col] = s;
        }
        cluster.sync();
        if (tid < D) {
            double s = 0.0;
#pragma unroll
            for (int r = 0; r < ECL; ++r) s += npart[r * D + tid];
            nrm[tid] = take_sqrt ? sqrt(s) : s;
        }
        cluster.sync();                                // nobody overwrites npart before everyone has read it
    };

    // Sweeps.  Columns are handled in 64 blocks of 2; a round pairs the blocks (tournament order, 63 rounds per
    // sweep) and a team of 16 lanes owns one pair of blocks = 4 columns.  The team forms the 4 x 4 Gram matrix of
    // its columns (partial over the local rows, exchanged through distributed shared memory: ONE cluster barrier
    // per round), then runs the three stages (0,1)(2,3) / (0,2)(1,3) / (0,3)(1,2) of rotations on the Gram matrix
    // itself -- in exact arithmetic the same rotations the column-by-column method would take -- and applies the six
    // rotations to its rows.  Every CTA sums the partials in the same order, so all take bit-identical decisions.
    // 4 lanes per team, 8 rows per lane: threads 0..127 move data, the rest only keep the barriers company
    constexpr int TL = 8, RPL = ESL_ROWS / TL;
    const int team16 = tid / TL, l16 = tid % TL;
    const bool mover = tid < 32 * TL;
    bool converged = false;
    int sweep = 0;
    for (; sweep < EIG_MAX_SWEEPS && !converged; ++sweep) {
        int big = 0;
        for (int round = 0; round < D / 2 - 1; ++round) {
            int col[4] = {0, 0, 0, 0};
            double x[RPL][4];
            if (mover) {
                int bp, bq;
                if (team16 == 0) { bp = D / 2 - 1; bq = round; }
                else { bp = (round + team16) % (D / 2 - 1); bq = (round - team16 + (D / 2 - 1)) % (D / 2 - 1); }
                col[0] = 2 * bp; col[1] = 2 * bp + 1; col[2] = 2 * bq; col[3] = 2 * bq + 1;
#pragma unroll
                for (int k = 0; k < 4; ++k)
#pragma unroll
                    for (int i = 0; i < RPL; ++i) x[i][k] = Gl[col[k] * ESL_LD + l16 + TL * i];
                double pg[10];                           // upper triangle of the partial Gram matrix
                int n = 0;
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int b = a; b < 4; ++b) {
                        double v = 0.0;
#pragma unroll
                        for (int i = 0; i < RPL; ++i) v = fma(x[i][a], x[i][b], v);
#pragma unroll
                        for (int m = 1; m < TL; m <<= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
                        pg[n++] = v;
                    }
                // lane l sends all ten values to CTA l
                if (l16 < ECL) {
                    double *dst = gpart_remote[l16 % ECL] + (round & 1) * (ECL * 32 * 10) + crank * 320 + team16;
#pragma unroll
                    for (int k = 0; k < 10; ++k) dst[k * 32] = pg[k];
                }
            }
            cluster.barrier_arrive();
            cluster.barrier_wait();
            // the six rotations of every team are worked out once, by one lane per team (warp 0), and broadcast
            if (tid < 32) {
                double g[4][4];
                const double *slot = gpart + (round & 1) * (ECL * 32 * 10) + tid;
                int n = 0;
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int b = a; b < 4; ++b) {
                        double v = 0.0;
#pragma unroll
                        for (int r = 0; r < ECL; ++r) v += slot[r * 320 + n * 32];
                        g[a][b] = g[b][a] = v;
                        ++n;
                    }
                double cc[6], ss[6];
                gram_stage<0, 1, 2, 3>(g, null_thr, tol2, cc[0], ss[0], cc[1], ss[1], big);
                gram_stage<0, 2, 1, 3>(g, null_thr, tol2, cc[2], ss[2], cc[3], ss[3], big);
                gram_stage<0, 3, 1, 2>(g, null_thr, tol2, cc[4], ss[4], cc[5], ss[5], big);
#pragma unroll
                for (int k = 0; k < 6; ++k) {
                    rotcs[tid * 12 + 2 * k] = cc[k];
                    rotcs[tid * 12 + 2 * k + 1] = ss[k];
                }
            }
            __syncthreads();
            double c[6], sn[6];
#pragma unroll
            for (int k = 0; k < 6; ++k) {
                c[k] = rotcs[(mover ? team16 : 0) * 12 + 2 * k];
                sn[k] = rotcs[(mover ? team16 : 0) * 12 + 2 * k + 1];
            }
            constexpr int RP[6] = {0, 2, 0, 1, 0, 1}, RQ[6] = {1, 3, 2, 3, 3, 2};
            if (mover) {
#pragma unroll
                for (int row = 0; row < RPL; ++row) {
#pragma unroll
                    for (int k = 0; k < 6; ++k) {
                        const double xp_ = x[row][RP[k]], xq_ = x[row][RQ[k]];
                        x[row][RP[k]] = c[k] * xp_ - sn[k] * xq_;
                        x[row][RQ[k]] = sn[k] * xp_ + c[k] * xq_;
                    }
                }
#pragma unroll
                for (int k = 0; k < 4; ++k)
#pragma unroll
                    for (int i = 0; i < RPL; ++i) Gl[col[k] * ESL_LD + l16 + TL * i] = x[i][k];
            }
            __syncthreads();                           // this round's rotations are visible to the next round's reads
        }
        converged = (__syncthreads_or(big) == 0);      // identical in every CTA: same Gram matrices everywhere
    }
    if (tid == 0 && crank == 0) {
        sweeps_out[h] = sweep;
        if (!converged) atomicOr(status, SQUAT_FLAG_NO_CONVERGE);
    }

    refresh_norms(true);                               // nrm = singular values of L = sqrt(mu + shift)
    if (tid < D) {
        const double mine = nrm[tid];
        int rk = 0;
        for (int j = 0; j < D; ++j) {
            const double o = nrm[j];
            rk += (o > mine) || (o == mine && j < tid);
        }
        rank[tid] = rk;
        if (crank == 0) {
            const double mu_out = mine * mine - shift;
            eigval[(long long)h * D + rk] = mu_out > 0.0 ? mu_out : 0.0;
        }
    }
    __syncthreads();
    for (int idx = tid; idx < D * ESL_ROWS; idx += ECT) {
        const int col = idx / ESL_ROWS, r = idx % ESL_ROWS;
        const double mu = nrm[col];
        const double v = mu > 0.0 ? Gl[col * ESL_LD + r] / mu : 0.0;
        eigvec[(long long)h * D * D + (long long)rank[col] * D + crank * ESL_ROWS + r] = v;
    }
    cluster.sync();                                    // no CTA exits while a peer may still write into it
}

// ------------------------------------------------------------------------------------- assemble
constexpr int ASM_THREADS = 512;
constexpr int ASM_LD = D + 1;

__global__ void __launch_bounds__(ASM_THREADS, 1) assemble_kernel(
    const double *__restrict__ eigval, const double *__restrict__ eigvec, int rank_r, double lambda, int g,
    float *__restrict__ Wt)
{
    extern __shared__ __align__(16) double sm[];
    double *A = sm;                         // A[row * ASM_LD + col]
    double *colv = sm + D * ASM_LD;         // column j before scaling
    double *lcol = colv + D;                // column j of L
    double *coef = lcol + D;                // s_i / (1 + s_i)
    const int h = blockIdx.x, tid = threadIdx.x;
    const double *V = eigvec + (long long)h * D * D;

    if (tid < D) {
        double mu = eigval[(long long)h * D + tid];
        if (!(mu > 0.0)) mu = 0.0;
        const double s = lambda * mu;
        coef[tid] = (tid < rank_r) ? s / (1.0 + s) : 0.0;
    }
    __syncthreads();
    // P_inv = I - sum_{i<r} coef_i v_i v_i^T, register-tiled: thread (ta, tb) owns rows 4 ta .. 4 ta + 3 and columns
    // 8 tb .. 8 tb + 7; the eigenvectors are staged 32 at a time in shared memory behind A
    {
        double *U = coef + D;                           // [32][D] staged eigenvectors
        const int ta = tid >> 4, tb = tid & 15;         // 32 x 16 tiles
        double acc[4][8];
#pragma unroll
        for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int y = 0; y < 8; ++y) acc[x][y] = (4 * ta + x == 8 * tb + y) ? 1.0 : 0.0;
        for (int i0 = 0; i0 < rank_r; i0 += 32) {
            const int ni = rank_r - i0 < 32 ? rank_r - i0 : 32;
            __syncthreads();
            for (int idx = tid; idx < ni * D; idx += ASM_THREADS) U[idx] = V[(long long)i0 * D + idx];
            __syncthreads();
            for (int i = 0; i < ni; ++i) {
                const double cf = -coef[i0 + i];
                double a[4], b[8];
#pragma unroll
                for (int x = 0; x < 4; x += 2) {
                    const double2 v = *reinterpret_cast<const double2 *>(U + i * D + 4 * ta + x);
                    a[x] = cf * v.x; a[x + 1] = cf * v.y;
                }
#pragma unroll
                for (int y = 0; y < 8; y += 2) {
                    const double2 v = *reinterpret_cast<const double2 *>(U + i * D + 8 * tb + y);
                    b[y] = v.x; b[y + 1] = v.y;
                }
#pragma unroll
                for (int x = 0; x < 4; ++x)
#pragma unroll
                    for (int y = 0; y < 8; ++y) acc[x][y] = fma(a[x], b[y], acc[x][y]);
            }
        }
#pragma unroll
        for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int y = 0; y < 8; ++y) A[(4 * ta + x) * ASM_LD + 8 * tb + y] = acc[x][y];
    }
    __syncthreads();
    // in-place LDL^T (right-looking): afterwards the strict lower triangle of A holds L
    for (int j = 0; j < D - 1; ++j) {
        if (tid > j && tid < D) {
            const double v = A[tid * ASM_LD + j];
            colv[tid] = v;
            lcol[tid] = v / A[j * ASM_LD + j];
        }
        __syncthreads();
        // trailing update (full square, both triangles kept); 2-D thread grid, no index division
        for (int i = j + 1 + (tid >> 5); i < D; i += ASM_THREADS / 32) {
            const double li = lcol[i];
            for (int k = j + 1 + (tid & 31); k < D; k += 32) A[i * ASM_LD + k] = fma(-li, colv[k], A[i * ASM_LD + k]);
        }
        if (tid > j && tid < D) A[tid * ASM_LD + j] = lcol[tid];
        __syncthreads();
    }
    // g > 1: block column t becomes L[rest, blk] * inverse(unit-lower diagonal block)
    if (g > 1) {
        const int T = D / g;
        for (int idx = tid; idx < D * (T - 1); idx += ASM_THREADS) {
            const int row = idx % D, t = idx / D;          // block t: columns [t*g, (t+1)*g)
            const int c0 = t * g;
            if (row < c0 + g) continue;
            double *x = A + row * ASM_LD + c0;
            for (int c = g - 2; c >= 0; --c) {
                double s = x[c];
                for (int cp = c + 1; cp < g; ++cp) s = fma(-x[cp], A[(c0 + cp) * ASM_LD + c0 + c], s);
                x[c] = s;
            }
        }
        __syncthreads();
    }
    // Wt[j][j'] = W[j'][j]: zero on and above the block diagonal
    float *out = Wt + (long long)h * D * D;
    for (int idx = tid; idx < D * D; idx += ASM_THREADS) {
        const int j = idx / D, jp = idx % D;
        const int blk_end = (j / g + 1) * g;
        out[idx] = (jp >= blk_end) ? (float)A[jp * ASM_LD + j] : 0.0f;
    }
}

}  // namespace

int squat_launch_gram(squat_subspace *s, const void *q, int dtype, int n_q_heads, int n_tokens,
                      long long stride_h, long long stride_t, cudaStream_t st)
{
    const int H = s->n_kv_heads, qpk = n_q_heads / H;
    const long long N = (long long)n_tokens * qpk;
    int chunks = s->gram_chunks_cap;
    long long rows_per_chunk = (N + chunks - 1) / chunks;
    rows_per_chunk = (rows_per_chunk + GRAM_ROWS - 1) / GRAM_ROWS * GRAM_ROWS;
    if (rows_per_chunk < 2 * GRAM_ROWS) rows_per_chunk = 2 * GRAM_ROWS;
    chunks = (int)((N + rows_per_chunk - 1) / rows_per_chunk);
    if (chunks < 1) chunks = 1;
    dim3 grid(chunks, H);
    if (dtype == SQUAT_BF16)
        gram_kernel<true><<<grid, GRAM_THREADS, 0, st>>>(q, n_tokens, qpk, stride_h, stride_t, (int)rows_per_chunk, s->gram_partial);
    else
        gram_kernel<false><<<grid, GRAM_THREADS, 0, st>>>(q, n_tokens, qpk, stride_h, stride_t, (int)rows_per_chunk, s->gram_partial);
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    gram_reduce_kernel<<<dim3(D * D / 256, H), 256, 0, st>>>(s->gram_partial, chunks, H, s->gram);
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return SQUAT_OK;
}

int squat_launch_eig(squat_subspace *s, cudaStream_t st)
{
    const size_t smem = sizeof(double) * (D * EIG_LD + D * ESL_LD + 2 * ECL * 32 * 10 + ECL * D + D + 32 * 12) + sizeof(int) * D;
    SQUAT_CUDA(cudaFuncSetAttribute(eig_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    eig_cluster_kernel<<<s->n_kv_heads * ECL, ECT, smem, st>>>(s->gram, s->eigval, s->eigvec, s->eig_sweeps, s->status);
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return SQUAT_OK;
}

int squat_launch_assemble(squat_subspace *s, int rank_r, double lambda, int block_g, cudaStream_t st)
{
    const size_t smem = sizeof(double) * (D * ASM_LD + 3 * D + 32 * D);
    SQUAT_CUDA(cudaFuncSetAttribute(assemble_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    assemble_kernel<<<s->n_kv_heads, ASM_THREADS, smem, st>>>(s->eigval, s->eigvec, rank_r, lambda, block_g, s->Wt);
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return SQUAT_OK;
}

// ------------------------------------------------------------------------- allocation-free Gram entry
// Scratch for squat_gram_static: the per-chunk partial Gram matrices live in this fixed array instead of
// memory obtained from cudaMalloc.  64 units of one d x d fp64 matrix = 8 MiB, held by every GPU that loads
// the library until the process exits.
namespace {
constexpr int GRAM_STATIC_MAX_UNITS = 64;            // n_kv_heads x row chunks
static __device__ __align__(256) double g_gram_static_scratch[(size_t)GRAM_STATIC_MAX_UNITS * D * D];
double *g_gram_static_ptr[64] = {nullptr};           // device address of the array, per device ordinal
}  // namespace

extern "C" int squat_gram_static(const void *q, int dtype, int n_q_heads, int n_kv_heads, int n_tokens,
                                 int head_dim, long long stride_h, long long stride_t, double *gram_out,
                                 void *stream)
{
    if (!q || !gram_out || (dtype != SQUAT_F32 && dtype != SQUAT_BF16)) return SQUAT_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(q) & 15u) || (reinterpret_cast<uintptr_t>(gram_out) & 15u)) return SQUAT_ERR_INVALID_ARG;
    if (n_q_heads <= 0 || n_kv_heads <= 0 || n_tokens <= 0) return SQUAT_ERR_INVALID_ARG;
    if (head_dim != D) return SQUAT_ERR_UNSUPPORTED;
    if (n_kv_heads > GRAM_STATIC_MAX_UNITS) return SQUAT_ERR_UNSUPPORTED;      // beyond the fixed scratch
    if (n_q_heads % n_kv_heads != 0) return SQUAT_ERR_SHAPE;
    const long long vec = dtype == SQUAT_BF16 ? 8 : 4;
    if (stride_t < D || stride_h < 0 || stride_t % vec || stride_h % vec) return SQUAT_ERR_INVALID_ARG;

    // set-up, once per device, with that device current: the array's name is only a host-side handle here;
    // kernels must be given the device address that cudaGetSymbolAddress reports
    int dev = 0;
    SQUAT_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return SQUAT_ERR_UNSUPPORTED;
    if (!g_gram_static_ptr[dev]) {
        double *ptr = nullptr;
        SQUAT_CUDA(cudaGetSymbolAddress((void **)&ptr, g_gram_static_scratch));
        g_gram_static_ptr[dev] = ptr;
    }
    double *partial = g_gram_static_ptr[dev];

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int H = n_kv_heads, qpk = n_q_heads / H;
    const long long N = (long long)n_tokens * qpk;
    int chunks = GRAM_STATIC_MAX_UNITS / H;                                   // >= 1
    long long rows_per_chunk = (N + chunks - 1) / chunks;
    rows_per_chunk = (rows_per_chunk + GRAM_ROWS - 1) / GRAM_ROWS * GRAM_ROWS;
    if (rows_per_chunk < 2 * GRAM_ROWS) rows_per_chunk = 2 * GRAM_ROWS;
    chunks = (int)((N + rows_per_chunk - 1) / rows_per_chunk);
    if (chunks < 1) chunks = 1;
    // every element the reduction reads is written by this call's first kernel, so nothing left in the
    // array by an earlier call is ever seen and nothing needs clearing
    dim3 grid(chunks, H);
    if (dtype == SQUAT_BF16)
        gram_kernel<true><<<grid, GRAM_THREADS, 0, st>>>(q, n_tokens, qpk, stride_h, stride_t, (int)rows_per_chunk, partial);
    else
        gram_kernel<false><<<grid, GRAM_THREADS, 0, st>>>(q, n_tokens, qpk, stride_h, stride_t, (int)rows_per_chunk, partial);
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    gram_reduce_kernel<<<dim3(D * D / 256, H), 256, 0, st>>>(partial, chunks, H, gram_out);
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return SQUAT_OK;
}

