// Step 1 with the block power method in place of the full eigen-decomposition (the accelerator the paper names in
// the comment on line 5 of Algorithm 1; the paper gives no steps, these are the textbook ones), all in fp64.
//
// Per KV head, from the Gram matrix M of the stacked prompt queries and a start block X0 [d, r]:
//     X <- orth(M X)   `iters` times     (orth = Cholesky QR: G = Y^T Y = L L^T, X = Y L^-T)
//     X <- orth(X)                        (a second pass: the first leaves X^T X = I only to eps * cond(Y)^2)
//     B = X^T M X,  N = I + lambda B
// and P^-1 = (I + lambda X B X^T)^-1 = I - X (I - N^-1) X^T = I - Z X^T with Z = X - X N^-1 (Woodbury with
// orthonormal X): X B X^T, the compression of M to the iterated subspace, stands where the full method has the
// rank-r truncation of M, and no eigen-decomposition of B is needed because P depends on span(X) only.  The kernel
// leaves the columns of X and of Z where the assembling kernel looks for its "right" and "left" vectors.
//
// A pivot of a Cholesky QR below 1e-13 of its diagonal entry marks a column that depends on the earlier ones (a start
// block or a Gram matrix of rank below r, or the zero columns that pad r to the kernel's block width): that column of
// X becomes zero and contributes nothing from then on.  One pass of Cholesky QR needs cond(M restricted to the block)
// well below 1e6.5; beyond that, directions are dropped and the count of kept columns (reported per head) says so.
//
// One CTA per head; X and Y are stored column by column with an odd stride, so that column dot products (lanes =
// different columns), products with M (lanes = different rows) and the per-row triangular solves (lanes = different
// rows) are all free of shared-memory bank conflicts.  No waiting on anything but __syncthreads.
#include "squat_internal.cuh"

namespace {

constexpr int D = SQUAT_D;
constexpr int PW_THREADS = 512;
constexpr int LDC = D + 1;                      // column stride of X and Y (doubles)
constexpr double PW_DROP = 1e-13;

template <int RP>
struct PowerLayout {
    static constexpr int LDG = RP + 1;                                         // row stride of G / L
    static constexpr size_t doubles = 2 * (size_t)RP * LDC + (size_t)RP * LDG + 2 * RP + 8;
};

// Y = M X: thread = rows (2 rp, 2 rp + 1) x column quads; M is symmetric, so row k of M holds column k
template <int RP>
__device__ __forceinline__ void pw_mult(const double *__restrict__ M, const double *Xt, double *Yt, int tid)
{
    constexpr int NQ = RP / 32;                 // column quads per thread
    const int rp = tid & 63, cs = tid >> 6;
    double acc[NQ][4][2];
#pragma unroll
    for (int u = 0; u < NQ; ++u)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[u][b][0] = acc[u][b][1] = 0.0;
#pragma unroll 4
    for (int k = 0; k < D; ++k) {
        const double2 m = __ldg(reinterpret_cast<const double2 *>(M + (size_t)k * D) + rp);
#pragma unroll
        for (int u = 0; u < NQ; ++u)
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const double x = Xt[(4 * (cs + 8 * u) + b) * LDC + k];
                acc[u][b][0] = fma(m.x, x, acc[u][b][0]);
                acc[u][b][1] = fma(m.y, x, acc[u][b][1]);
            }
    }
#pragma unroll
    for (int u = 0; u < NQ; ++u)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            double *y = Yt + (4 * (cs + 8 * u) + b) * LDC + 2 * rp;
            y[0] = acc[u][b][0];
            y[1] = acc[u][b][1];
        }
}

// G[i][j] = add_identity * (i == j) + scale * sum_row At[i][row] Bt[j][row]
template <int RP>
__device__ __forceinline__ void pw_gram(const double *At, const double *Bt, double *G, double scale, double ident, int tid)
{
    constexpr int NJ = RP * RP / PW_THREADS;    // 2 (RP = 32) or 8 (RP = 64) columns j per thread
    constexpr int LDG = PowerLayout<RP>::LDG;
    const int i = tid % RP, j0 = (tid / RP) * NJ;
    double acc[NJ];
#pragma unroll
    for (int b = 0; b < NJ; ++b) acc[b] = 0.0;
#pragma unroll 4
    for (int row = 0; row < D; ++row) {
        const double a = At[i * LDC + row];
#pragma unroll
        for (int b = 0; b < NJ; ++b) acc[b] = fma(a, Bt[(j0 + b) * LDC + row], acc[b]);
    }
#pragma unroll
    for (int b = 0; b < NJ; ++b) G[i * LDG + j0 + b] = scale * acc[b] + ((i == j0 + b) ? ident : 0.0);
}

// In-place Cholesky G = L L^T of the lower triangle by one warp (left-looking; lane = rows lane, lane + 32).  A pivot
// at or below drop * (its diagonal entry) zeroes the column: L[.][j] = 0, inv[j] = 0.  Returns the kept columns.
template <int RP>
__device__ __forceinline__ int pw_chol(double *G, double *inv, double drop, int lane)
{
    constexpr int NR = RP / 32;
    constexpr int LDG = PowerLayout<RP>::LDG;
    int kept = 0;
    for (int j = 0; j < RP; ++j) {
        double v[NR];
#pragma unroll
        for (int u = 0; u < NR; ++u) {
            const int i = lane + 32 * u;
            double s0 = 0.0, s1 = 0.0;
            if (i >= j) {
                const double *gi = G + i * LDG, *gj = G + j * LDG;
                int k = 0;
                for (; k + 1 < j; k += 2) { s0 = fma(gi[k], gj[k], s0); s1 = fma(gi[k + 1], gj[k + 1], s1); }
                if (k < j) s0 = fma(gi[k], gj[k], s0);
                v[u] = gi[j] - (s0 + s1);
            } else {
                v[u] = 0.0;
            }
        }
        const double g0 = G[j * LDG + j];
        double pv;                              // the pivot: v of row j, held by lane j % 32 (no dynamic register index)
        if (NR == 1) {
            pv = __shfl_sync(0xffffffffu, v[0], j & 31);
        } else {
            const double p0 = __shfl_sync(0xffffffffu, v[0], j & 31), p1 = __shfl_sync(0xffffffffu, v[NR - 1], j & 31);
            pv = (j < 32) ? p0 : p1;
        }
        const bool ok = pv > drop * g0 && pv > 0.0;
        const double ljj = ok ? sqrt(pv) : 0.0;
        const double iv = ok ? 1.0 / ljj : 0.0;
        kept += ok ? 1 : 0;
        __syncwarp();
#pragma unroll
        for (int u = 0; u < NR; ++u) {
            const int i = lane + 32 * u;
            if (i > j) G[i * LDG + j] = v[u] * iv;
            else if (i == j) { G[j * LDG + j] = ljj; inv[j] = iv; }
        }
        __syncwarp();
    }
    return kept;
}

// rows of  Dst = Src L^-T  (forward substitution, one thread per row; Dst may be Src)
template <int RP>
__device__ __forceinline__ void pw_solve_forward(const double *Src, double *Dst, const double *L, const double *inv, int row)
{
    constexpr int LDG = PowerLayout<RP>::LDG;
    for (int j = 0; j < RP; ++j) {
        const double *lj = L + j * LDG;
        double s0 = Src[j * LDC + row], s1 = 0.0;
        int k = 0;
        for (; k + 1 < j; k += 2) { s0 = fma(-Dst[k * LDC + row], lj[k], s0); s1 = fma(-Dst[(k + 1) * LDC + row], lj[k + 1], s1); }
        if (k < j) s0 = fma(-Dst[k * LDC + row], lj[k], s0);
        Dst[j * LDC + row] = (s0 + s1) * inv[j];
    }
}

// rows of  Dst <- Dst L^-1  (backward substitution, in place)
template <int RP>
__device__ __forceinline__ void pw_solve_backward(double *Dst, const double *L, const double *inv, int row)
{
    constexpr int LDG = PowerLayout<RP>::LDG;
    for (int j = RP - 1; j >= 0; --j) {
        double s0 = Dst[j * LDC + row], s1 = 0.0;
        int k = j + 1;
        for (; k + 1 < RP; k += 2) { s0 = fma(-Dst[k * LDC + row], L[k * LDG + j], s0); s1 = fma(-Dst[(k + 1) * LDC + row], L[(k + 1) * LDG + j], s1); }
        if (k < RP) s0 = fma(-Dst[k * LDC + row], L[k * LDG + j], s0);
        Dst[j * LDC + row] = (s0 + s1) * inv[j];
    }
}

template <int RP>
__global__ void __launch_bounds__(PW_THREADS, 1) power_kernel(
    const double *__restrict__ gram, const double *__restrict__ start, long long start_stride_h, int r, int iters,
    double lambda, double *__restrict__ vec_out, int *__restrict__ kept_out)
{
    extern __shared__ __align__(16) double psm[];
    constexpr int LDG = PowerLayout<RP>::LDG;
    double *A = psm;                            // [RP][LDC]
    double *Bf = A + RP * LDC;                  // [RP][LDC]
    double *G = Bf + RP * LDC;                  // [RP][LDG]
    double *inv = G + RP * LDG;                 // [RP]
    int *kept_sm = reinterpret_cast<int *>(inv + 2 * RP);
    const int h = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    const double *M = gram + (size_t)h * D * D;
    const double *X0 = start + (size_t)h * start_stride_h;

    for (int idx = tid; idx < RP * D; idx += PW_THREADS) {
        const int c = idx / D, k = idx % D;
        A[c * LDC + k] = (c < r) ? X0[(size_t)k * r + c] : 0.0;
    }
    __syncthreads();
    double *X = A, *Y = Bf;
    // iters passes of X <- orth(M X), then one more orth(X) (for iters = 0 that makes two passes over X0)
    for (int it = (iters == 0 ? -1 : 0); it <= iters; ++it) {
        double *T;                              // what gets orthonormalised in this pass
        if (it >= 0 && it < iters) {
            pw_mult<RP>(M, X, Y, tid);
            __syncthreads();
            T = Y;
        } else {
            T = X;
        }
        pw_gram<RP>(T, T, G, 1.0, 0.0, tid);
        __syncthreads();
        if (tid < 32) {
            const int kept = pw_chol<RP>(G, inv, PW_DROP, lane);
            if (lane == 0) *kept_sm = kept;
        }
        __syncthreads();
        if (tid < D) pw_solve_forward<RP>(T, T, G, inv, tid);
        __syncthreads();
        if (T == Y) { double *t = X; X = Y; Y = t; }
    }
    if (tid == 0) kept_out[h] = *kept_sm;
    // B = X^T (M X),  N = I + lambda B = L L^T,  Z = X - X N^-1
    pw_mult<RP>(M, X, Y, tid);
    __syncthreads();
    pw_gram<RP>(X, Y, G, lambda, 1.0, tid);
    __syncthreads();
    if (tid < 32) pw_chol<RP>(G, inv, 0.0, lane);
    __syncthreads();
    if (tid < D) {
        pw_solve_forward<RP>(X, Y, G, inv, tid);
        pw_solve_backward<RP>(Y, G, inv, tid);
    }
    __syncthreads();
    // rows [0, r) of the output: columns of X (right vectors); rows [64, 64 + r): columns of Z (left vectors)
    double *out = vec_out + (size_t)h * D * D;
    for (int idx = tid; idx < r * D; idx += PW_THREADS) {
        const int c = idx / D, k = idx % D;
        const double x = X[c * LDC + k];
        out[(size_t)c * D + k] = x;
        out[(size_t)(64 + c) * D + k] = x - Y[c * LDC + k];
    }
}

}  // namespace

int squat_launch_power(squat_subspace *s, const double *start, long long start_stride_h, int rank_r, int iters,
                       double lambda, cudaStream_t st)
{
    if (rank_r <= 32) {
        const size_t smem = PowerLayout<32>::doubles * sizeof(double);
        SQUAT_CUDA(cudaFuncSetAttribute(power_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        power_kernel<32><<<s->n_kv_heads, PW_THREADS, smem, st>>>(s->gram, start, start_stride_h, rank_r, iters, lambda,
                                                               s->eigvec, s->eig_sweeps);
    } else {
        const size_t smem = PowerLayout<64>::doubles * sizeof(double);
        SQUAT_CUDA(cudaFuncSetAttribute(power_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        power_kernel<64><<<s->n_kv_heads, PW_THREADS, smem, st>>>(s->gram, start, start_stride_h, rank_r, iters, lambda,
                                                               s->eigvec, s->eig_sweeps);
    }
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return SQUAT_OK;
}
