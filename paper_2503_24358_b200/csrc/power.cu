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
// One CTA of 256 threads per head; X and Y are stored column by column with an odd stride, so that column dot products (lanes =
// different columns), products with M (lanes = different rows) and the per-row triangular solves (lanes = different
// rows) are all free of shared-memory bank conflicts.  No waiting on anything but __syncthreads.
#include "squat_internal.cuh"

namespace {

constexpr int D = SQUAT_D;
constexpr int PW_THREADS = 256;
constexpr int LDC = D + 1;                      // column stride of X and Y (doubles)
constexpr double PW_DROP = 1e-13;

template <int RP>
struct PowerLayout {
    static constexpr int LDG = RP + 1;                                         // row stride of G / L
    static constexpr bool M_SHARED = RP <= 32;                                 // M beside X, Y fits in shared memory
    static constexpr size_t small = 2 * (size_t)RP * LDC + (size_t)RP * LDG + RP + 8;   // X, Y, G, inv, misc
    static constexpr size_t doubles = small + (M_SHARED ? (size_t)D * D : 0);
};

// Y = M X: thread = rows 4 rq .. 4 rq + 3 x 8 columns (warp-uniform); M is symmetric, so row k of M holds column k.
// With 32 columns four warps cover them and the other four take the second half of the sum over k, added after a
// barrier; with 64 columns every warp has its own 8.
template <int RP, bool MS>
__device__ __forceinline__ void pw_mult(const double *__restrict__ M, const double *Xt, double *Yt, int tid)
{
    constexpr int KS = (RP == 32) ? 2 : 1;      // parts of the k range
    const int rq = tid & 31, w = tid >> 5;
    const int c0 = 8 * (w % (RP / 8)), part = w / (RP / 8);
    double acc[8][4];
#pragma unroll
    for (int b = 0; b < 8; ++b)
#pragma unroll
        for (int a = 0; a < 4; ++a) acc[b][a] = 0.0;
    const int k_lo = part * (D / KS), k_hi = k_lo + D / KS;
#pragma unroll 2
    for (int k = k_lo; k < k_hi; ++k) {
        const double2 *mp = reinterpret_cast<const double2 *>(M + (size_t)k * D) + 2 * rq;
        const double2 m01 = MS ? mp[0] : __ldg(mp);                 // MS: M is a shared-memory copy
        const double2 m23 = MS ? mp[1] : __ldg(mp + 1);
        const double m[4] = {m01.x, m01.y, m23.x, m23.y};
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            const double x = Xt[(c0 + b) * LDC + k];
#pragma unroll
            for (int a = 0; a < 4; ++a) acc[b][a] = fma(m[a], x, acc[b][a]);
        }
    }
    if (part == 0) {
#pragma unroll
        for (int b = 0; b < 8; ++b)
#pragma unroll
            for (int a = 0; a < 4; ++a) Yt[(c0 + b) * LDC + 4 * rq + a] = acc[b][a];
    }
    if (KS == 2) {
        __syncthreads();
        if (part == 1) {
#pragma unroll
            for (int b = 0; b < 8; ++b)
#pragma unroll
                for (int a = 0; a < 4; ++a) Yt[(c0 + b) * LDC + 4 * rq + a] += acc[b][a];
        }
    }
}

// G[i][j] = add_identity * (i == j) + scale * sum_row At[i][row] Bt[j][row]
template <int RP>
__device__ __forceinline__ void pw_gram(const double *At, const double *Bt, double *G, double scale, double ident, int tid)
{
    constexpr int NJ = RP * RP / PW_THREADS;    // 4 (RP = 32) or 16 (RP = 64) columns j per thread
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

// 1 / sqrt(x) for a positive normal x: exponent split off (x = s * 4^n with s in [1, 4)), single-precision seed, two
// Newton steps in double precision (2^-22 -> 2^-44 -> beyond 2^-53), exponent put back.
__device__ __forceinline__ double pw_rsqrt(double x)
{
    const int hi = __double2hiint(x), lo = __double2loint(x);
    const int e2 = (((hi >> 20) & 0x7ff) - 1023) & ~1;
    const double s = __hiloint2double(hi - (e2 << 20), lo);
    double y = (double)rsqrtf((float)s);
    const double hs = 0.5 * s;
    y = y * fma(-hs * y, y, 1.5);
    y = y * fma(-hs * y, y, 1.5);
    return __hiloint2double(__double2hiint(y) - ((e2 >> 1) << 20), __double2loint(y));
}

// In-place Cholesky G = L L^T of the lower triangle by one warp, left-looking in panels of 8 columns; lane = rows
// lane (and lane + 32).  A panel's entries live in registers: first the contributions of the columns to its left (a
// loop over them, rows of L read from shared memory), then 8 elimination steps with the pivot row's values passed by
// shuffles (a fully unrolled 32-column variant with the whole row in registers measured twice as slow).  A pivot at
// or below drop * (the diagonal entry it started from) zeroes the column: L[.][j] = 0, inv[j] = 0.  Returns the
// number of kept columns.
template <int RP>
__device__ __noinline__ int pw_chol(double *G, double *inv, double drop, int lane)
{
    constexpr int NR = RP / 32;
    constexpr int LDG = PowerLayout<RP>::LDG;
    int kept = 0;
#pragma unroll 1
    for (int jb = 0; jb < RP; jb += 8) {
        double a[NR][8], g0[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) g0[c] = G[(jb + c) * LDG + jb + c];
#pragma unroll
        for (int u = 0; u < NR; ++u)
#pragma unroll
            for (int c = 0; c < 8; ++c) a[u][c] = G[(lane + 32 * u) * LDG + jb + c];
#pragma unroll 2
        for (int k = 0; k < jb; ++k) {
            double lj[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) lj[c] = G[(jb + c) * LDG + k];
#pragma unroll
            for (int u = 0; u < NR; ++u) {
                const double lik = G[(lane + 32 * u) * LDG + k];
#pragma unroll
                for (int c = 0; c < 8; ++c) a[u][c] = fma(-lik, lj[c], a[u][c]);
            }
        }
        const int us = jb >> 5;                                     // which of the lane's rows the pivot rows are
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int jj = jb + j;
            const double mine = (NR == 1 || us == 0) ? a[0][j] : a[NR - 1][j];
            const double pv = __shfl_sync(0xffffffffu, mine, jj & 31);
            const bool ok = pv > drop * g0[j] && pv > 1e-290;
            const double iv = ok ? pw_rsqrt(pv) : 0.0;
            double l[NR];
#pragma unroll
            for (int u = 0; u < NR; ++u) {
                const int i = lane + 32 * u;
                l[u] = i > jj ? a[u][j] * iv : 0.0;
                a[u][j] = i > jj ? l[u] : (i == jj ? pv * iv : a[u][j]);
            }
            if (lane == 0) inv[jj] = iv;
            kept += ok ? 1 : 0;
#pragma unroll
            for (int c = j + 1; c < 8; ++c) {
                const double lsrc = (NR == 1 || us == 0) ? l[0] : l[NR - 1];
                const double lc = __shfl_sync(0xffffffffu, lsrc, (jb + c) & 31);
#pragma unroll
                for (int u = 0; u < NR; ++u) a[u][c] = fma(-l[u], lc, a[u][c]);
            }
        }
#pragma unroll
        for (int u = 0; u < NR; ++u)
#pragma unroll
            for (int c = 0; c < 8; ++c)
                if (lane + 32 * u >= jb + c) G[(lane + 32 * u) * LDG + jb + c] = a[u][c];
        __syncwarp();
    }
    return kept;
}

// rows of  Dst = Src L^-T  (forward substitution, one thread per row, 8 columns at a time in registers; Dst may be Src)
template <int RP>
__device__ __noinline__ void pw_solve_forward(const double *Src, double *Dst, const double *L, const double *inv, int row)
{
    constexpr int LDG = PowerLayout<RP>::LDG;
#pragma unroll 1
    for (int jb = 0; jb < RP; jb += 8) {
        double y[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) y[c] = Src[(jb + c) * LDC + row];
#pragma unroll 2
        for (int k = 0; k < jb; ++k) {
            const double xk = Dst[k * LDC + row];
#pragma unroll
            for (int c = 0; c < 8; ++c) y[c] = fma(-xk, L[(jb + c) * LDG + k], y[c]);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const double x = y[j] * inv[jb + j];
            y[j] = x;
#pragma unroll
            for (int c = j + 1; c < 8; ++c) y[c] = fma(-x, L[(jb + c) * LDG + jb + j], y[c]);
        }
#pragma unroll
        for (int c = 0; c < 8; ++c) Dst[(jb + c) * LDC + row] = y[c];
    }
}

// rows of  Dst <- Dst L^-1  (backward substitution, in place, same blocking)
template <int RP>
__device__ __noinline__ void pw_solve_backward(double *Dst, const double *L, const double *inv, int row)
{
    constexpr int LDG = PowerLayout<RP>::LDG;
#pragma unroll 1
    for (int jb = RP - 8; jb >= 0; jb -= 8) {
        double y[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) y[c] = Dst[(jb + c) * LDC + row];
#pragma unroll 2
        for (int k = jb + 8; k < RP; ++k) {                         // the later columns, already solved
            const double xk = Dst[k * LDC + row];
#pragma unroll
            for (int c = 0; c < 8; ++c) y[c] = fma(-xk, L[k * LDG + jb + c], y[c]);
        }
#pragma unroll
        for (int j = 7; j >= 0; --j) {
            const double x = y[j] * inv[jb + j];
            y[j] = x;
#pragma unroll
            for (int c = 0; c < j; ++c) y[c] = fma(-x, L[(jb + j) * LDG + jb + c], y[c]);
        }
#pragma unroll
        for (int c = 0; c < 8; ++c) Dst[(jb + c) * LDC + row] = y[c];
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
    int *kept_sm = reinterpret_cast<int *>(inv + RP);
    const int h = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    constexpr bool MS = PowerLayout<RP>::M_SHARED;
    const double *M = gram + (size_t)h * D * D;
    const double *Mu = M;                       // what the multiplications read
    if (MS) {
        double *Msm = psm + PowerLayout<RP>::small;
        for (int idx = tid; idx < D * D / 2; idx += PW_THREADS)
            reinterpret_cast<double2 *>(Msm)[idx] = __ldg(reinterpret_cast<const double2 *>(M) + idx);
        Mu = Msm;
    }
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
            pw_mult<RP, MS>(Mu, X, Y, tid);
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
    pw_mult<RP, MS>(Mu, X, Y, tid);
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
