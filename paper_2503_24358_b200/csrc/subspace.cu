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
#include <type_traits>
#include <utility>
#include "squat_internal.cuh"

namespace {

constexpr int D = SQUAT_D;

// ------------------------------------------------------------------------------------- Gram
// M = Qc^T Qc on the fp64 tensor-core path (mma.sync m8n8k4, fp64 operands and accumulators: products of bf16 or
// fp32 inputs are exact in fp64).  M is symmetric: of the 16 x 16 grid of 8 x 8 tiles only the 136 tiles on or above
// the diagonal are computed, 17 per warp, 8 warps per CTA.  The A fragment of tile row i (A[m][k] = Q[token k][8 i + m])
// and the B fragment of tile column i (B[k][n] = Q[token k][8 i + n]) are the same register, so a warp loads one
// fragment per 8-channel group and 4-token step and feeds it to every tile that touches the group.
constexpr int GRAM_THREADS = 256;
constexpr int GRAM_ROWS = 32;                  // token rows staged in shared memory per step
constexpr int GRAM_LDR = D + 4;                // row stride (doubles): 4 tokens x 8 channels of a fragment hit 32 distinct words
constexpr int GRAM_TILES_PER_WARP = 17;
constexpr int GRAM_CTAS_PER_SM = 2;

// u-th tile of the upper triangle, row by row: (ti, tj), ti <= tj
template <int U>
struct GramTile {
    static constexpr int row()
    {
        int u = U, ti = 0, len = 16;
        while (u >= len) { u -= len; --len; ++ti; }
        return ti;
    }
    static constexpr int ti = row();
    static constexpr int tj = ti + (U - (ti * 16 - ti * (ti - 1) / 2));
};

__device__ __forceinline__ void dmma_m8n8k4(double &c0, double &c1, double a, double b)
{
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                 : "+d"(c0), "+d"(c1) : "d"(a), "d"(b));
}

template <int W, int... N>
__device__ __forceinline__ void gram_warp_step(double (&acc)[GRAM_TILES_PER_WARP][2], const double (&F)[16],
                                               std::integer_sequence<int, N...>)
{
    (dmma_m8n8k4(acc[N][0], acc[N][1], F[GramTile<GRAM_TILES_PER_WARP * W + N>::ti], F[GramTile<GRAM_TILES_PER_WARP * W + N>::tj]), ...);
}

template <int W, int... N>
__device__ __forceinline__ void gram_warp_store(const double (&acc)[GRAM_TILES_PER_WARP][2], double *out, int lane,
                                                std::integer_sequence<int, N...>)
{
    // C fragment: thread holds row lane / 4, columns 2 (lane % 4) and 2 (lane % 4) + 1 of the tile
    ((*reinterpret_cast<double2 *>(out + (GramTile<GRAM_TILES_PER_WARP * W + N>::ti * 8 + (lane >> 2)) * D +
                                   GramTile<GRAM_TILES_PER_WARP * W + N>::tj * 8 + 2 * (lane & 3)) = make_double2(acc[N][0], acc[N][1])), ...);
}

template <bool BF16, int W>
__device__ __forceinline__ void gram_warp_body(const double *rows, double (&acc)[GRAM_TILES_PER_WARP][2], int lane)
{
    const double *base = rows + (lane & 3) * GRAM_LDR + (lane >> 2);
#pragma unroll 2
    for (int k0 = 0; k0 < GRAM_ROWS; k0 += 4) {
        double F[16];
#pragma unroll
        for (int g = 0; g < 16; ++g) F[g] = base[k0 * GRAM_LDR + g * 8];
        gram_warp_step<W>(acc, F, std::make_integer_sequence<int, GRAM_TILES_PER_WARP>{});
    }
}

template <bool BF16>
__global__ void __launch_bounds__(GRAM_THREADS, GRAM_CTAS_PER_SM) gram_kernel(
    const void *__restrict__ q, int n_tokens, int q_per_kv, long long stride_h, long long stride_t,
    int rows_per_chunk, double *__restrict__ partial /* [chunks, H, D, D] */)
{
    __shared__ __align__(16) double rows[GRAM_ROWS * GRAM_LDR];
    const int h = blockIdx.y, chunk = blockIdx.x, H = gridDim.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long N = (long long)n_tokens * q_per_kv;
    const long long row_lo = (long long)chunk * rows_per_chunk;
    long long row_hi = row_lo + rows_per_chunk;
    if (row_hi > N) row_hi = N;

    double acc[GRAM_TILES_PER_WARP][2];
#pragma unroll
    for (int n = 0; n < GRAM_TILES_PER_WARP; ++n) acc[n][0] = acc[n][1] = 0.0;

    // Staging: a thread moves pairs of neighbouring channels (4 bytes of bf16, 8 of fp32), so that a warp's
    // 16-byte stores of the converted pairs fall on consecutive words.  The global loads of step s + 1 are
    // issued before the arithmetic of step s, so their latency is hidden.
    constexpr int NPAIR = GRAM_ROWS * (D / 2) / GRAM_THREADS;          // 16
    using raw_t = typename std::conditional<BF16, uint32_t, uint2>::type;
    raw_t pre[NPAIR];
    // A thread's pairs of one step sit in rows r0 + rr0 + 4 it of the stack (rr0 = thread / 64) at a fixed channel pair.
    // Row n of the stack is token n mod n_tokens of query head n / n_tokens of the KV head: (head, token) of the
    // thread's first row are divided out once and then carried from row to row and from step to step (fetch is called
    // for consecutive steps), so the loop holds no division.
    static_assert(GRAM_THREADS / (D / 2) == 4 && NPAIR * 4 == GRAM_ROWS, "four rows per pass of the CTA over a step");
    const int c2 = threadIdx.x % (D / 2), rr0 = threadIdx.x / (D / 2);
    int q_next = 0, t_next = 0;                                     // query head and token of row (next r0) + rr0
    if (row_lo < row_hi) {
        const long long n0 = row_lo + rr0;
        q_next = (int)(n0 / n_tokens);
        t_next = (int)(n0 - (long long)q_next * n_tokens);
    }
    auto fetch = [&](long long r0) {
        int qh = q_next, t = t_next;
#pragma unroll
        for (int it = 0; it < NPAIR; ++it) {
            const long long n = r0 + rr0 + 4 * it;
            pre[it] = raw_t{};
            if (n < row_hi) {
                const long long off = ((long long)h * q_per_kv + qh) * stride_h + (long long)t * stride_t + c2 * 2;
                if constexpr (BF16) pre[it] = __ldg(reinterpret_cast<const uint32_t *>(reinterpret_cast<const __nv_bfloat16 *>(q) + off));
                else pre[it] = __ldg(reinterpret_cast<const uint2 *>(reinterpret_cast<const float *>(q) + off));
            }
            t += 4;
            while (t >= n_tokens) { t -= n_tokens; ++qh; }
        }
        q_next = qh;                                                // = (head, token) of row r0 + GRAM_ROWS + rr0
        t_next = t;
    };
    if (row_lo < row_hi) fetch(row_lo);
    for (long long r0 = row_lo; r0 < row_hi; r0 += GRAM_ROWS) {
        __syncthreads();
#pragma unroll
        for (int it = 0; it < NPAIR; ++it) {
            const int idx = threadIdx.x + it * GRAM_THREADS;
            const int rr = idx / (D / 2), c2 = idx % (D / 2);
            double2 v;
            if constexpr (BF16) { v.x = (double)bf16lo_to_f32(pre[it]); v.y = (double)bf16hi_to_f32(pre[it]); }
            else { v.x = (double)__uint_as_float(pre[it].x); v.y = (double)__uint_as_float(pre[it].y); }
            *reinterpret_cast<double2 *>(&rows[rr * GRAM_LDR + c2 * 2]) = v;
        }
        __syncthreads();
        if (r0 + GRAM_ROWS < row_hi) fetch(r0 + GRAM_ROWS);
        switch (warp) {
        case 0: gram_warp_body<BF16, 0>(rows, acc, lane); break;
        case 1: gram_warp_body<BF16, 1>(rows, acc, lane); break;
        case 2: gram_warp_body<BF16, 2>(rows, acc, lane); break;
        case 3: gram_warp_body<BF16, 3>(rows, acc, lane); break;
        case 4: gram_warp_body<BF16, 4>(rows, acc, lane); break;
        case 5: gram_warp_body<BF16, 5>(rows, acc, lane); break;
        case 6: gram_warp_body<BF16, 6>(rows, acc, lane); break;
        default: gram_warp_body<BF16, 7>(rows, acc, lane); break;
        }
    }
    double *out = partial + ((long long)chunk * H + h) * D * D;
    constexpr auto seq = std::make_integer_sequence<int, GRAM_TILES_PER_WARP>{};
    switch (warp) {
    case 0: gram_warp_store<0>(acc, out, lane, seq); break;
    case 1: gram_warp_store<1>(acc, out, lane, seq); break;
    case 2: gram_warp_store<2>(acc, out, lane, seq); break;
    case 3: gram_warp_store<3>(acc, out, lane, seq); break;
    case 4: gram_warp_store<4>(acc, out, lane, seq); break;
    case 5: gram_warp_store<5>(acc, out, lane, seq); break;
    case 6: gram_warp_store<6>(acc, out, lane, seq); break;
    default: gram_warp_store<7>(acc, out, lane, seq); break;
    }
}

// Sums the per-chunk partials in a fixed order and mirrors the upper tiles: gram[h] full symmetric.  One thread takes four
// neighbouring elements of a row of one of the 136 stored tiles (two 16-byte loads per chunk, all chunks' loads
// independent) and writes them and, for a tile above the diagonal, their mirror images.
constexpr int GRED_UNITS = 136 * 16;           // 136 tiles x 8 rows x 2 halves of a row
constexpr int GRED_THREADS = 128;
__global__ void __launch_bounds__(GRED_THREADS) gram_reduce_kernel(const double *__restrict__ partial, int chunks, int H, double *__restrict__ gram)
{
    const int h = blockIdx.y;
    const int unit = blockIdx.x * GRED_THREADS + threadIdx.x;
    if (unit >= GRED_UNITS) return;
    int u = unit >> 4, ti = 0, len = 16;       // u-th tile of the upper triangle, row by row
    while (u >= len) { u -= len; --len; ++ti; }
    const int tj = ti + u;
    const int a = 8 * ti + ((unit >> 1) & 7), b = 8 * tj + 4 * (unit & 1);
    const double *src = partial + (long long)h * D * D + a * D + b;
    double2 s0 = make_double2(0.0, 0.0), s1 = s0;
    for (int c = 0; c < chunks; ++c) {
        const double2 v0 = *reinterpret_cast<const double2 *>(src + (long long)c * H * D * D);
        const double2 v1 = *reinterpret_cast<const double2 *>(src + (long long)c * H * D * D + 2);
        s0.x += v0.x; s0.y += v0.y; s1.x += v1.x; s1.y += v1.y;
    }
    double *g = gram + (long long)h * D * D;
    *reinterpret_cast<double2 *>(g + a * D + b) = s0;
    *reinterpret_cast<double2 *>(g + a * D + b + 2) = s1;
    if (ti != tj) {
        g[(b + 0) * D + a] = s0.x;
        g[(b + 1) * D + a] = s0.y;
        g[(b + 2) * D + a] = s1.x;
        g[(b + 3) * D + a] = s1.y;
    }
}

// ------------------------------------------------------------------------------------- eigen
constexpr int EIG_MAX_SWEEPS = 40;

// Eigen-decomposition of M: Cholesky M + shift I = L L^T, then one-sided (Hestenes) Jacobi on the columns of L.
// L has the square root of M's condition number and L^T L is much closer to diagonal than M^2, which cuts the
// sweeps (14 -> 10 on the 4096-token workload).  The shift (1e-12 of the trace) keeps the factorisation defined
// for rank-deficient M and is subtracted from the eigenvalues at the end; eigenvectors are unaffected by it.
// Rotations are skipped below 1e-14 relative; a sweep that applied none above that level is the last.
//
// One head is worked on by a cluster of 4 CTAs (4 SMs per head instead of 1; a 32-head layer then occupies 128
// of the 148 SMs).  The 128 columns form 8 blocks of 16, and every CTA holds two blocks with ALL their rows, so a
// rotation of two columns held by the same CTA needs no communication at all: a team of 16 lanes owns the pair
// (8 rows per lane), the dot product is a 4-step shuffle reduction, and rounds inside a CTA are separated by a
// barrier among the 8 working warps only.
// A sweep is
//   one intra phase   15 rounds that pair the columns inside each held block (8 + 8 pairs per round), then
//   7 block rounds    of 16 rounds each that pair every column of one held block with every column of the other;
//                     after each block round one block of every CTA moves to another CTA (schedule below), so
//                     that over the 7 block rounds every block has met every other one.
// So the CTAs talk 7 times per sweep instead of once per round.  After a block round every column sits in some
// team's registers and is written straight into the spare buffer of its next holder (through distributed shared
// memory if that is a peer); one cluster barrier per move publishes the data and guarantees that nobody is a block
// round behind, which is what makes the spare buffers free.  The squared column norms ride along with the block:
// they are refreshed from the data at the start of a sweep and updated by each rotation in between
// (alpha' = alpha - t gamma, beta' = beta + t gamma), so a round reduces one dot product, not three.
// The Cholesky factorisation is done redundantly by each CTA on a full copy (it is a small part of the time).
namespace cg = cooperative_groups;
constexpr int ECL = 4;                       // CTAs per cluster
constexpr int ECT = 512;                     // threads per CTA: 16 warps = 16 column pairs per round
constexpr int BW = 16;                       // columns per block
constexpr int BLD = D + 2;                   // column stride inside a block buffer (doubles)
constexpr int BLK_DOUBLES = BW * BLD + BW;   // 16 columns and their 16 squared norms
// Block schedule of a sweep: 7 block rounds, each pairing the two blocks a CTA holds, such that every two of the 8
// blocks meet exactly once (a 1-factorisation of K8 found by a randomised search; of the candidates tried, the one
// that needed the fewest sweeps on the benchmark's Gram matrices) while only ONE block per CTA changes
// hands between consecutive rounds -- the minimum, since two blocks that have met must part.  Move m (after
// block round m): bit c of MOVE_KEEP1[m] says that CTA c keeps its slot-1 block (else its slot-0 block); the other
// one goes to CTA (MOVE_TO[m] >> 2c) & 3, where it becomes slot 1.  The schedule is positional, so it covers all
// pairs from whatever arrangement the previous sweep left.
__constant__ unsigned char MOVE_KEEP1[7] = {0x5, 0xb, 0x9, 0xd, 0xe, 0x5, 0x5};
__constant__ unsigned char MOVE_TO[7] = {0x1e, 0x4b, 0xb1, 0x4e, 0x39, 0x8d, 0x1e};
constexpr unsigned BLK_BYTES = BLK_DOUBLES * (unsigned)sizeof(double);
static_assert(GRAM_TILES_PER_WARP * (GRAM_THREADS / 32) == 136, "the warps share the upper triangle evenly");
static_assert(D / BW == 2 * ECL, "two blocks per CTA");
static_assert(BLK_BYTES % 16 == 0, "bulk copies move 16-byte units");

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
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

// 1/x for a normal double: hardware seed (about 20 bits), two Newton steps y <- y + y (1 - x y)
__device__ __forceinline__ double rcp_nr(double x)
{
    double y;
    asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(x));
    y = fma(y, fma(-x, y, 1.0), y);
    return fma(y, fma(-x, y, 1.0), y);
}

__device__ __forceinline__ void named_bar_sync(int id, int count) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory"); }

// One Jacobi rotation of a column pair (P, Q) held in registers by a team of 16 lanes (both halves of a warp work
// on different pairs): lane l owns rows l, l + 16, ..., l + 112.  alpha, beta are the (cached) squared norms, kept by
// every lane; gamma = P . Q is reduced here.  New P = c P - s Q, new Q = s P + c Q with the angle that makes them
// orthogonal (tan 2theta = 2 gamma / (beta - alpha), |theta| <= pi/4), from two reciprocal square roots.  A pair
// already orthogonal to 1e-14 relative, or numerically null twice over, is left alone (returns 0); otherwise
// returns 1, or 3 when the pair started above the convergence level.
constexpr int TLN = 16;                      // lanes per team
constexpr int TROWS = D / TLN;               // rows per lane of a team: 2 tl + 32 i and 2 tl + 1 + 32 i, i < TROWS / 2
__device__ __forceinline__ void load_col(double (&x)[TROWS], const double *col, int tl)
{
#pragma unroll
    for (int i = 0; i < TROWS / 2; ++i) {
        const double2 v = *reinterpret_cast<const double2 *>(col + 2 * tl + 2 * TLN * i);
        x[2 * i] = v.x;
        x[2 * i + 1] = v.y;
    }
}
__device__ __forceinline__ void store_col(double *col, const double (&x)[TROWS], int tl)
{
#pragma unroll
    for (int i = 0; i < TROWS / 2; ++i) *reinterpret_cast<double2 *>(col + 2 * tl + 2 * TLN * i) = make_double2(x[2 * i], x[2 * i + 1]);
}
__device__ __forceinline__ int rotate_regs(double (&xp)[TROWS], double (&xq)[TROWS], double &alpha, double &beta, double null_thr)
{
    double g0 = 0.0, g1 = 0.0;
#pragma unroll
    for (int i = 0; i < TROWS; i += 2) { g0 = fma(xp[i], xq[i], g0); g1 = fma(xp[i + 1], xq[i + 1], g1); }
    double gam = g0 + g1;
#pragma unroll
    for (int m = TLN / 2; m >= 1; m >>= 1) gam += __shfl_xor_sync(0xffffffffu, gam, m);
    const double g2 = gam * gam, ab = alpha * beta;
    if (!((alpha > null_thr || beta > null_thr) && g2 > 1e-28 * ab)) return 0;      // uniform over the team
    const double diff = beta - alpha;
    const double inv_r = rsqrt_nr(fma(diff, diff, 4.0 * g2));
    const double hc = fma(0.5 * fabs(diff), inv_r, 0.5);              // (1 + cos 2theta)/2 = c^2, in [1/2, 1]
    const double inv_c = rsqrt_nr(hc);
    const double c = hc * inv_c;
    const double sm = gam * inv_r * inv_c;
    const double s = diff < 0.0 ? -sm : sm;
    const double t = s * inv_c;                                       // tan(theta)
#pragma unroll
    for (int i = 0; i < TROWS; ++i) {
        const double p = xp[i], q = xq[i];
        xp[i] = c * p - s * q;
        xq[i] = s * p + c * q;
    }
    alpha -= t * gam;
    beta += t * gam;
    return g2 > 1e-14 * ab ? 3 : 1;
}

__global__ void __cluster_dims__(ECL, 1, 1) __launch_bounds__(ECT, 1) eig_cluster_kernel(
    const double *__restrict__ gram, double *__restrict__ eigval, double *__restrict__ eigvec,
    int *__restrict__ sweeps_out, unsigned *__restrict__ status)
{
    cg::cluster_group cluster = cg::this_cluster();
    const int crank = (int)cluster.block_rank();
    extern __shared__ __align__(16) double sm[];
    double *blk = sm;                                  // [2 buffers][2 slots][BLK_DOUBLES]: the held blocks and the spare
    double *nall = blk + 4 * BLK_DOUBLES;              // [ECL][32] final column norms of the whole cluster
    double *lcol = nall + ECL * 32;                    // [2][D] column of L being eliminated (double-buffered)
    double *red = lcol + 2 * D;                        // [16] per-warp partial sums
    int *flags = reinterpret_cast<int *>(red + 16);    // [ECL] "rotated above the convergence level" per CTA
    const int h = blockIdx.x / ECL, tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const double *M = gram + (long long)h * D * D;

    // Cholesky factorisation M + shift I = L L^T with the matrix in REGISTERS: thread (lane, warp) owns the
    // elements (row lane + 32 i, column warp + 16 k), i < 4, k < 8; only those on or below the diagonal are used.
    // Step j: the warp that owns column j gets the pivot by a shuffle, scales its column and publishes it in shared
    // memory; after ONE barrier (the column buffer alternates) every thread subtracts the rank-1 term from its
    // elements.  Columns of the two blocks this CTA starts with go straight into the block buffers:
    // positions crank (slot 0) and 7 - crank (slot 1).
    double a[4][8];
    double tr = 0.0;
#pragma unroll
    for (int k = 0; k < 8; ++k)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = lane + 32 * i, c = warp + 16 * k;
            a[i][k] = M[c * D + r];                    // M is symmetric: read along the contiguous direction
            if (r == c) tr += a[i][k];
        }
    tr = warp_sum(tr);
    if (lane == 0) red[warp] = tr;
    __syncthreads();
    double trace = 0.0;
#pragma unroll
    for (int w = 0; w < 16; ++w) trace += red[w];
    const double shift = trace > 0.0 ? 1e-12 * trace : 1e-300;       // M + shift I = L L^T
#pragma unroll
    for (int k = 0; k < 8; ++k)
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (lane + 32 * i == warp + 16 * k) a[i][k] += shift;
#pragma unroll
    for (int kj = 0; kj < 8; ++kj) {
        const int slot = kj == crank ? 0 : (kj == 2 * ECL - 1 - crank ? 1 : -1);
#pragma unroll 1
        for (int wj = 0; wj < 16; ++wj) {
            const int j = 16 * kj + wj;
            double *lc = lcol + (j & 1) * D;
            if (warp == wj) {
                double piv = __shfl_sync(0xffffffffu, a[kj >> 1][kj], j & 31);
                piv = piv > 0.0 ? piv : shift;
                const double inv = rsqrt_nr(piv);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int r = lane + 32 * i;
                    const double l = r > j ? a[i][kj] * inv : (r == j ? piv * inv : 0.0);
                    lc[r] = l;
                    if (slot >= 0) blk[slot * BLK_DOUBLES + wj * BLD + r] = l;
                }
            }
            __syncthreads();
            double lr[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) lr[i] = lc[lane + 32 * i];
#pragma unroll
            for (int k = kj; k < 8; ++k) {
                const int c = warp + 16 * k;
                if (c > j) {                           // warp-uniform
                    const double lcc = lc[c];
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (32 * i + 31 >= 16 * k) a[i][k] = fma(-lr[i], lcc, a[i][k]);
                }
            }
        }
    }
    __syncthreads();
    const double null_thr = 4.0 * shift;
    cluster.sync();                                    // every CTA of the cluster is running before anybody writes into it

    // squared norms of the 32 held columns, from the data: warp w takes columns w and w + 16
    auto refresh_norms = [&](double *cur) {
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            double *col = cur + k * BLK_DOUBLES + warp * BLD;
            double s = 0.0;
#pragma unroll
            for (int i = 0; i < 4; ++i) { const double v = col[lane + 32 * i]; s = fma(v, v, s); }
            s = warp_sum(s);
            if (lane == 0) cur[k * BLK_DOUBLES + BW * BLD + warp] = s;
        }
        __syncthreads();
    };

    int cur_buf = 0;                                   // which buffer holds the blocks
    bool converged = false;
    int sweep = 0;
    for (; sweep < EIG_MAX_SWEEPS && !converged; ++sweep) {
        int big = 0;
        double *cur = blk + cur_buf * 2 * BLK_DOUBLES;
        refresh_norms(cur);
        // Pairs are worked on by 16 teams of 16 lanes (warps 0-7); they keep in step through a barrier of their own.
        const int team = tid / TLN, tl = tid % TLN;
        constexpr int TEAM_THREADS = 16 * TLN;
        // intra phase: round-robin of the 16 columns of a block; teams 0-7 on slot 0, teams 8-15 on slot 1
        if (tid < TEAM_THREADS) {
            double *b = cur + (team >> 3) * BLK_DOUBLES, *nb = b + BW * BLD;
            const int t = team & 7;
            for (int round = 0; round < BW - 1; ++round) {
                int p, q;
                if (t == 0) { p = BW - 1; q = round; }
                else { p = (round + t) % (BW - 1); q = (round - t + (BW - 1)) % (BW - 1); }
                double xp[TROWS], xq[TROWS];
                load_col(xp, b + p * BLD, tl);
                load_col(xq, b + q * BLD, tl);
                double alpha = nb[p], beta = nb[q];
                const int did = rotate_regs(xp, xq, alpha, beta, null_thr);
                if (did) {
                    store_col(b + p * BLD, xp, tl);
                    store_col(b + q * BLD, xq, tl);
                    if (tl == 0) { nb[p] = alpha; nb[q] = beta; }
                }
                big |= did >> 1;
                named_bar_sync(1, TEAM_THREADS);
            }
        }
        __syncthreads();
        for (int br = 0; br < 2 * ECL - 1; ++br) {
            cur = blk + cur_buf * 2 * BLK_DOUBLES;
            // block round: team t keeps column t of slot 0 in registers and meets column (t + round) mod 16 of slot 1
            if (tid < TEAM_THREADS) {
                double *b0 = cur, *b1 = cur + BLK_DOUBLES, *n0 = b0 + BW * BLD, *n1 = b1 + BW * BLD;
                double xa[TROWS], xb[TROWS];
                load_col(xa, b0 + team * BLD, tl);
                double alpha = n0[team], beta = 0.0;
                for (int round = 0; round < BW; ++round) {
                    const int q = (team + round) & (BW - 1);
                    load_col(xb, b1 + q * BLD, tl);
                    beta = n1[q];
                    const int did = rotate_regs(xa, xb, alpha, beta, null_thr);
                    if (did && round < BW - 1) {
                        store_col(b1 + q * BLD, xb, tl);
                        if (tl == 0) n1[q] = beta;
                    }
                    big |= did >> 1;
                    named_bar_sync(1, TEAM_THREADS);
                }
                // Move the blocks on.  After the last round every column sits in some team's registers (column `team`
                // of slot 0 and column team + 15 mod 16 of slot 1).  Each CTA keeps one of its two blocks (it becomes
                // slot 0 of the other buffer: plain stores) and sends the other to a peer (slot 1 of the peer's other
                // buffer: stores through distributed shared memory), as the schedule says.  That buffer is free: its
                // owner left it when it began this block round.
                const bool keep1 = (MOVE_KEEP1[br] >> crank) & 1;
                double *kept_home = blk + ((cur_buf ^ 1) * 2 + 0) * BLK_DOUBLES;
                double *sent_home = cluster.map_shared_rank(blk + ((cur_buf ^ 1) * 2 + 1) * BLK_DOUBLES, (MOVE_TO[br] >> (2 * crank)) & 3);
                double *d0 = keep1 ? sent_home : kept_home, *d1 = keep1 ? kept_home : sent_home;
                const int ql = (team + BW - 1) & (BW - 1);
                store_col(d0 + team * BLD, xa, tl);
                store_col(d1 + ql * BLD, xb, tl);
                if (tl == 0) { d0[BW * BLD + team] = alpha; d1[BW * BLD + ql] = beta; }
            }
            if (br == 2 * ECL - 2) {
                // the sweep is the last one if no CTA of the cluster rotated a pair from above the convergence level
                big = __syncthreads_or(big);
                if (tid < ECL) *cluster.map_shared_rank(&flags[crank], tid) = big ? 1 : 0;
            }
            cluster.sync();                            // blocks (and flags) have arrived; nobody is behind by a block round
            cur_buf ^= 1;
        }
        int any = 0;
#pragma unroll
        for (int r = 0; r < ECL; ++r) any |= flags[r];  // rewritten only after seven more cluster barriers
        converged = any == 0;
    }
    if (tid == 0 && crank == 0) {
        sweeps_out[h] = sweep;
        if (!converged) atomicOr(status, SQUAT_FLAG_NO_CONVERGE);
    }

    // singular values of L = sqrt(mu + shift) are the column norms; rank them over the whole cluster
    double *cur = blk + cur_buf * 2 * BLK_DOUBLES;
    refresh_norms(cur);
    if (tid < 32) {
        const double n2 = cur[(tid >> 4) * BLK_DOUBLES + BW * BLD + (tid & 15)];
        const double nv = sqrt(n2);
#pragma unroll
        for (int r = 0; r < ECL; ++r) *cluster.map_shared_rank(&nall[crank * 32 + tid], r) = nv;
    }
    cluster.sync();
    for (int k = 0; k < 2; ++k) {                      // warp w writes held columns w (slot 0) and w (slot 1)
        const int id = crank * 32 + k * BW + warp;
        const double mine = nall[id];
        int rk = 0;
        for (int j = lane; j < D; j += 32) {
            const double o = nall[j];
            rk += (o > mine) || (o == mine && j < id);
        }
#pragma unroll
        for (int m = 16; m >= 1; m >>= 1) rk += __shfl_xor_sync(0xffffffffu, rk, m);
        const double *col = cur + k * BLK_DOUBLES + warp * BLD;
        const double inv = mine > 0.0 ? 1.0 / mine : 0.0;
#pragma unroll
        for (int i = 0; i < 4; ++i)
            eigvec[(long long)h * D * D + (long long)rk * D + lane + 32 * i] = col[lane + 32 * i] * inv;
        if (lane == 0) {
            const double mu_out = mine * mine - shift;
            eigval[(long long)h * D + rk] = mu_out > 0.0 ? mu_out : 0.0;
        }
    }
    cluster.sync();                                    // no CTA exits while a peer may still write into it
}

// ------------------------------------------------------------------------------------- assemble
constexpr int ASM_THREADS = 512;
constexpr int ASM_LD = D + 1;

__global__ void __launch_bounds__(ASM_THREADS, 1) assemble_kernel(
    const double *__restrict__ eigval, const double *__restrict__ eigvec, int rank_r, double lambda, int g,
    float *__restrict__ Wt, int left_rows)
{
    // left_rows = 0: P_inv = I - sum_i s_i/(1+s_i) v_i v_i^T from eigen-pairs (rows i of eigvec, eigval).
    // left_rows > 0: P_inv = I - sum_i z_i x_i^T with x_i = row i and z_i = row left_rows + i of eigvec (block power build).
    extern __shared__ __align__(16) double sm[];
    double *A = sm;                         // A[row * ASM_LD + col]
    double *colv = sm + D * ASM_LD;         // [2 parities][l, v][D]: column j of L and of the matrix, as published
    double *coef = colv + 4 * D;            // s_i / (1 + s_i)
    const int h = blockIdx.x, tid = threadIdx.x;
    const double *V = eigvec + (long long)h * D * D;

    if (tid < D) {
        double mu = eigval[(long long)h * D + tid];
        if (!(mu > 0.0)) mu = 0.0;
        const double s = lambda * mu;
        coef[tid] = (tid < rank_r) ? (left_rows > 0 ? 1.0 : s / (1.0 + s)) : 0.0;
    }
    __syncthreads();
    // The matrix lives in REGISTERS from here to the end of the factorisation: thread (lane, warp) owns the elements
    // (row lane + 32 i, column warp + 16 k), i < 4, k < 8; only those on or below the diagonal are used.
    const int warp = tid >> 5, lane = tid & 31;
    double a[4][8];
    // P_inv = I - sum_{i<r} coef_i v_i v_i^T; the eigenvectors are staged 32 at a time in shared memory
    {
        double *U = coef + D;                           // [32][D] staged eigenvectors (right vectors)
        double *UL = left_rows > 0 ? U + 32 * D : U;    // [32][D] staged left vectors
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int k = 0; k < 8; ++k) a[i][k] = (lane + 32 * i == warp + 16 * k) ? 1.0 : 0.0;
        for (int i0 = 0; i0 < rank_r; i0 += 32) {
            const int ni = rank_r - i0 < 32 ? rank_r - i0 : 32;
            __syncthreads();
            for (int idx = tid; idx < ni * D; idx += ASM_THREADS) U[idx] = V[(long long)i0 * D + idx];
            if (left_rows > 0)
                for (int idx = tid; idx < ni * D; idx += ASM_THREADS) UL[idx] = V[(long long)(left_rows + i0) * D + idx];
            __syncthreads();
            for (int e = 0; e < ni; ++e) {
                const double cf = -coef[i0 + e];
                double vr[4], vc[8];
#pragma unroll
                for (int i = 0; i < 4; ++i) vr[i] = cf * UL[e * D + lane + 32 * i];
#pragma unroll
                for (int k = 0; k < 8; ++k) vc[k] = U[e * D + warp + 16 * k];
#pragma unroll
                for (int k = 0; k < 8; ++k)
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (32 * i + 31 >= 16 * k) a[i][k] = fma(vr[i], vc[k], a[i][k]);
            }
        }
    }
    __syncthreads();
    // LDL^T (right-looking), afterwards the strict lower triangle holds L.  Step j: the warp that owns column j gets
    // the pivot d_j by a shuffle and publishes v = column j and l = v / d_j in shared memory; after ONE barrier (the
    // buffers alternate) every thread subtracts l_r v_c from its elements.
    {
        double *pub = colv;                             // [2 parities][l, v][D], overlays colv, lcol and more
#pragma unroll
        for (int kj = 0; kj < 8; ++kj) {
#pragma unroll 1
            for (int wj = 0; wj < 16; ++wj) {
                const int j = 16 * kj + wj;
                double *lp = pub + (j & 1) * 2 * D, *vp = lp + D;
                if (warp == wj) {
                    const double d = __shfl_sync(0xffffffffu, a[kj >> 1][kj], j & 31);
                    const double inv = rcp_nr(d);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int r = lane + 32 * i;
                        const double v = a[i][kj], l = v * inv;
                        if (r > j) { lp[r] = l; vp[r] = v; a[i][kj] = l; }
                    }
                }
                __syncthreads();
                double lr[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) lr[i] = lp[lane + 32 * i];     // rows <= j hold stale values: only feed unused elements
#pragma unroll
                for (int k = kj; k < 8; ++k) {
                    const int c = warp + 16 * k;
                    if (c > j) {                        // warp-uniform
                        const double vc = vp[c];
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            if (32 * i + 31 >= 16 * k) a[i][k] = fma(-lr[i], vc, a[i][k]);
                    }
                }
            }
        }
    }
    float *out = Wt + (long long)h * D * D;
    if (g == 1) {
        // Wt[j][j'] = W[j'][j] = L[j'][j] below the diagonal, zero on and above it: straight from the registers
#pragma unroll
        for (int k = 0; k < 8; ++k)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int r = lane + 32 * i, c = warp + 16 * k;
                out[c * D + r] = (r > c) ? (float)a[i][k] : 0.0f;
            }
        return;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 8; ++k)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = lane + 32 * i, c = warp + 16 * k;
            if (r > c) A[r * ASM_LD + c] = a[i][k];
        }
    __syncthreads();
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
    gram_reduce_kernel<<<dim3(GRED_UNITS / GRED_THREADS, H), GRED_THREADS, 0, st>>>(s->gram_partial, chunks, H, s->gram);
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return SQUAT_OK;
}

int squat_launch_eig(squat_subspace *s, cudaStream_t st)
{
    const size_t smem = sizeof(double) * (4 * BLK_DOUBLES + ECL * 32 + 2 * D + 16) + sizeof(int) * ECL;
    SQUAT_CUDA(cudaFuncSetAttribute(eig_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    eig_cluster_kernel<<<s->n_kv_heads * ECL, ECT, smem, st>>>(s->gram, s->eigval, s->eigvec, s->eig_sweeps, s->status);
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return SQUAT_OK;
}

int squat_launch_assemble(squat_subspace *s, int rank_r, double lambda, int block_g, int left_rows, int exact_blocks, cudaStream_t st)
{
    const size_t smem = sizeof(double) * (D * ASM_LD + 5 * D + 64 * D);
    SQUAT_CUDA(cudaFuncSetAttribute(assemble_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    assemble_kernel<<<s->n_kv_heads, ASM_THREADS, smem, st>>>(s->eigval, s->eigvec, rank_r, lambda, block_g, s->Wt, left_rows);
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return squat_launch_pack_update_matrices(s->Wt, s->Wimg, s->n_kv_heads, exact_blocks, s->exact_blocks, st);
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
    gram_reduce_kernel<<<dim3(GRED_UNITS / GRED_THREADS, H), GRED_THREADS, 0, st>>>(partial, chunks, H, gram_out);
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return SQUAT_OK;
}

