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
// One CTA of 256 threads per head.  The two kinds of products (M X and the Gram matrices Y^T Y, X^T (M X)) run on the
// FP64 tensor path (mma.sync m8n8k4), which has the throughput of the FP64 FMA path on this part but needs a third of
// the shared-memory reads and far fewer issue slots.  X and Y are stored column by column with a stride of d + 4
// doubles, M (for r <= 32, where it fits beside them) row by row with the same stride: the 8 x 4 operand fragments
// then fall on distinct banks, and the per-row triangular solves (lanes = consecutive rows) are conflict-free with any
// stride.  No waiting on anything but __syncthreads.
#include "squat_internal.cuh"

namespace {

constexpr int D = SQUAT_D;
constexpr int PW_THREADS = 256;
constexpr int LDC = D + 4;                      // column stride of X and Y (doubles): tensor-operation fragments (8 columns x 4 rows) fall on distinct banks
constexpr int LDM = D + 4;                      // row stride of the shared-memory copy of M, for the same reason
constexpr double PW_DROP = 1e-13;

template <int RP>
struct PowerLayout {
    static constexpr int LDG = RP + 1;                                         // row stride of G / L
    static constexpr bool M_SHARED = RP <= 32;                                 // M beside X, Y fits in shared memory
    static constexpr size_t small = 2 * (size_t)RP * LDC + (size_t)RP * LDG + RP + 8;   // X, Y, G, inv, misc
    static constexpr size_t doubles = small + (M_SHARED ? (size_t)D * LDM : 0);
};

// D += A B on the FP64 tensor path: A 8 x 4 (lane holds A[lane / 4][lane % 4]), B 4 x 8 (lane holds B[lane % 4][lane / 4]),
// D 8 x 8 (lane holds D[lane / 4][2 (lane % 4)] and the element to its right)
__device__ __forceinline__ void pw_dmma(double &c0, double &c1, double a, double b)
{
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                 : "+d"(c0), "+d"(c1) : "d"(a), "d"(b));
}

// Y = M X: a warp owns 16 rows (two 8-row tiles) x all RP columns; per 4 values of k it loads two fragments of M and
// RP / 8 of X and issues RP / 4 tensor operations.  M is symmetric; MS: M is the padded shared-memory copy (row stride
// LDM), else it is read from global memory (row stride D).
template <int RP, bool MS>
__device__ __forceinline__ void pw_mult(const double *__restrict__ M, const double *Xt, double *Yt, int tid)
{
    constexpr int NC = RP / 8;                  // column tiles
    constexpr int LD = MS ? LDM : D;
    const int warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    double acc[2][NC][2];
#pragma unroll
    for (int r = 0; r < 2; ++r)
#pragma unroll
        for (int c = 0; c < NC; ++c) acc[r][c][0] = acc[r][c][1] = 0.0;
    const double *ma = M + (size_t)(16 * warp + g) * LD + t;
    const double *xb = Xt + g * LDC + t;
#pragma unroll 2
    for (int k0 = 0; k0 < D; k0 += 4) {
        const double a0 = MS ? ma[k0] : __ldg(ma + k0);
        const double a1 = MS ? ma[8 * LD + k0] : __ldg(ma + 8 * LD + k0);
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            const double b = xb[8 * c * LDC + k0];
            pw_dmma(acc[0][c][0], acc[0][c][1], a0, b);
            pw_dmma(acc[1][c][0], acc[1][c][1], a1, b);
        }
    }
#pragma unroll
    for (int r = 0; r < 2; ++r)
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            double *y = Yt + (8 * c + 2 * t) * LDC + 16 * warp + 8 * r + g;
            y[0] = acc[r][c][0];
            y[LDC] = acc[r][c][1];
        }
}

// G[i][j] = ident * (i == j) + scale * sum_row At[i][row] Bt[j][row]: a warp owns one 8-row tile of G and RP * RP / 512
// of its 8-column tiles
template <int RP>
__device__ __forceinline__ void pw_gram(const double *At, const double *Bt, double *G, double scale, double ident, int tid)
{
    constexpr int LDG = PowerLayout<RP>::LDG;
    constexpr int NT = RP / 8;                  // tiles per side
    constexpr int NC = NT * NT / (PW_THREADS / 32);     // column tiles per warp: 2 (RP = 32) or 8 (RP = 64)
    const int warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int ti = (warp * NC) / NT, tj0 = (warp * NC) % NT;
    double acc[NC][2];
#pragma unroll
    for (int c = 0; c < NC; ++c) acc[c][0] = acc[c][1] = 0.0;
    const double *pa = At + (8 * ti + g) * LDC + t;
    const double *pb = Bt + (8 * tj0 + g) * LDC + t;
#pragma unroll 2
    for (int k0 = 0; k0 < D; k0 += 4) {
        const double a = pa[k0];
#pragma unroll
        for (int c = 0; c < NC; ++c) pw_dmma(acc[c][0], acc[c][1], a, pb[8 * c * LDC + k0]);
    }
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        const int i = 8 * ti + g, j = 8 * (tj0 + c) + 2 * t;
        G[i * LDG + j] = scale * acc[c][0] + (i == j ? ident : 0.0);
        G[i * LDG + j + 1] = scale * acc[c][1] + (i == j + 1 ? ident : 0.0);
    }
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
            *reinterpret_cast<double2 *>(Msm + (idx / (D / 2)) * LDM + 2 * (idx % (D / 2))) = __ldg(reinterpret_cast<const double2 *>(M) + idx);
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
