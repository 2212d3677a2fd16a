// Key quantization with error feedback for small subspace ranks: the same function Quant of Algorithm 1 with the
// update of Eq. (3), run through the rank-r form of the update matrices instead of the dense triangle.
//
// For element-wise updates (g = 1) the matrix W of Prop. 1 / Lemma 3 is semiseparable: with v_j the j-th row of
// V_r (the top-r right singular vectors, d x r) and S = lambda * diag(sigma_i^2),
//     W[j'][j] = v_j' . c_j   for j' > j,     c_j = -(I_r + S G_j)^-1 S v_j^T,     G_j = sum_{j' > j} v_j'^T v_j'
// (the Woodbury identity of the footnote to Prop. 4, applied to the trailing block P[j+1:, j+1:] = I + V S V^T of
// S1: B_t H_t = -P22^-1 P21).  So instead of d - j - 1 multiply-adds per channel a token carries a state s in R^r:
//     x_j = k_j + v_j . s          (the corrected value of channel j)
//     s  += e_j c_j                (after rounding channel j with error e_j)
// -- 2 r multiply-adds per channel, 2 r d per key vector, against d (d - 1) / 2 for the dense triangle: cheaper for
// r < (d - 1) / 4.  Built for r <= 8 (tables padded with zeros), where the whole update fits the FP32 pipes with no
// hand-over to the tensor cores and no tensor-memory limit on the warps in flight.
//
// Mapping.  lane = token, two tokens per lane (two spans of 32 consecutive tokens per warp: two groups for G = 32,
// the two halves of one group for G = 64, half a group for G = 128 where two warps pair up through shared memory
// and a named barrier).  The per-head table (d rows of [v_j | c_j], 8 KB) sits in shared memory and is read with
// broadcast 16-byte loads, each serving both tokens of every lane.  The rounding arithmetic is the dense kernel's
// (keys.cu), operation for operation.
#include "squat_internal.cuh"
#include <cuda_fp16.h>

namespace {

constexpr int D = SQUAT_D;
constexpr int R = SQUAT_LOWRANK_MAX_R;     // 8
constexpr int ROW = 2 * R;                 // floats per channel row of the table: v_j | c_j
constexpr int BLK = 32;
constexpr int NBLK = D / BLK;
constexpr int LR_WARPS = 8;
constexpr int LR_THREADS = LR_WARPS * 32;
constexpr int LR_CTAS_PER_SM = 3;          // 80 registers per thread: 24 warps per SM
constexpr float kMagic = 12582912.0f;      // 1.5 * 2^23

typedef unsigned long long u64;

__device__ __forceinline__ u64 pack2(float lo, float hi)
{
    u64 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ float lo_of(u64 v) { return __uint_as_float((unsigned)(v & 0xffffffffull)); }
__device__ __forceinline__ float hi_of(u64 v) { return __uint_as_float((unsigned)(v >> 32)); }
__device__ __forceinline__ u64 ffma2(u64 a, u64 b, u64 c)
{
    u64 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
// NaN-propagating reductions: a NaN key shows up in the stored scale and raises SQUAT_FLAG_NONFINITE
__device__ __forceinline__ float warp_min(float x)
{
    float r;
    asm volatile("redux.sync.min.NaN.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ float warp_max(float x)
{
    float r;
    asm volatile("redux.sync.max.NaN.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ float min_nan(float a, float b)
{
    float r;
    asm("min.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ float max_nan(float a, float b)
{
    float r;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}
// correctly rounded rng / L for L = 3 or 15 (as in keys.cu)
template <int BITS>
__device__ __forceinline__ float div_by_levels(float rng)
{
    constexpr float L = float((1 << BITS) - 1);
    constexpr float invL = 1.0f / L;
    const float q = __fmul_rn(rng, invL);
    const float r = __fmaf_rn(-L, q, rng);
    return __fmaf_rn(r, invL, q);
}

// ------------------------------------------------------------------------------------------ the per-head tables
// One CTA per head, thread j = channel j, everything fp64.  With sq_i = sqrt(S_i):
//     c_j = -S^1/2 (I + S^1/2 G_j S^1/2)^-1 S^1/2 v_j^T
// -- the symmetric form of (I + S G_j)^-1 S, whose matrix is positive definite with eigenvalues >= 1, solved by a
// Cholesky factorisation held in the thread's registers.
__global__ void __launch_bounds__(D) lowrank_table_kernel(const double *__restrict__ eigval, const double *__restrict__ eigvec,
                                                          int r, double lambda, float *__restrict__ table)
{
    __shared__ double Vs[R][D];            // Vs[i][j] = v_j[i] = component j of eigenvector i
    const int h = blockIdx.x, j = threadIdx.x;
    const double *vec = eigvec + (long long)h * D * D;
    for (int i = 0; i < R; ++i) Vs[i][j] = i < r ? vec[(long long)i * D + j] : 0.0;
    __syncthreads();
    double sq[R], A[R][R];
#pragma unroll
    for (int a = 0; a < R; ++a) {
        const double mu = a < r ? eigval[(long long)h * D + a] : 0.0;
        sq[a] = sqrt(fmax(lambda * mu, 0.0));
#pragma unroll
        for (int b = 0; b < R; ++b) A[a][b] = 0.0;
    }
    for (int jp = j + 1; jp < D; ++jp) {
#pragma unroll
        for (int a = 0; a < R; ++a)
#pragma unroll
            for (int b = 0; b <= a; ++b) A[a][b] = fma(Vs[a][jp], Vs[b][jp], A[a][b]);
    }
#pragma unroll
    for (int a = 0; a < R; ++a)
#pragma unroll
        for (int b = 0; b <= a; ++b) A[a][b] = sq[a] * sq[b] * A[a][b] + (a == b ? 1.0 : 0.0);
    // Cholesky A = L L^T (lower, in place)
#pragma unroll
    for (int c = 0; c < R; ++c) {
#pragma unroll
        for (int k = 0; k < c; ++k) A[c][c] = fma(-A[c][k], A[c][k], A[c][c]);
        A[c][c] = sqrt(A[c][c]);
        const double inv = 1.0 / A[c][c];
#pragma unroll
        for (int a = c + 1; a < R; ++a) {
#pragma unroll
            for (int k = 0; k < c; ++k) A[a][c] = fma(-A[a][k], A[c][k], A[a][c]);
            A[a][c] *= inv;
        }
    }
    double y[R];
#pragma unroll
    for (int a = 0; a < R; ++a) {               // L z = S^1/2 v_j
        double t = sq[a] * Vs[a][j];
#pragma unroll
        for (int k = 0; k < a; ++k) t = fma(-A[a][k], y[k], t);
        y[a] = t / A[a][a];
    }
#pragma unroll
    for (int a = R - 1; a >= 0; --a) {          // L^T y = z
        double t = y[a];
#pragma unroll
        for (int k = a + 1; k < R; ++k) t = fma(-A[k][a], y[k], t);
        y[a] = t / A[a][a];
    }
    float *row = table + ((long long)h * D + j) * ROW;
#pragma unroll
    for (int a = 0; a < R; ++a) {
        row[a] = (float)Vs[a][j];
        row[R + a] = (float)(-sq[a] * y[a]);
    }
}

// ------------------------------------------------------------------------------------------ the quantizer
struct LrParams {
    const float *table;       // [H, d, ROW]
    const void *k;
    long long sb, sh, st;     // element strides of k
    unsigned char *codes;
    void *scales, *zeros;
    long long osb, osh;       // output strides in tokens
    int groups_per_bh;        // T / G
    int spans_per_head;       // 32-token spans per head: B * T / 32
    int team_tasks;           // per head: tasks of one team (1 warp, or 2 for G = 128)
    unsigned *status;
#ifdef SQUAT_CHECKED
    SqExtent x_k, x_codes, x_scales, x_zeros, x_table;    // what the caller's tensors and the handle's tables span
#endif
};

template <bool BF16>
struct Raw16 {                // 16 channels of one token
    uint4 v[BF16 ? 2 : 4];
};
template <bool BF16>
__device__ __forceinline__ void load16(Raw16<BF16> &r, const void *row, int chan)
{
    if (BF16) {
        const uint4 *q = reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(row) + chan);
#pragma unroll
        for (int i = 0; i < 2; ++i) r.v[i] = __ldg(q + i);
    } else {
        const uint4 *q = reinterpret_cast<const uint4 *>(reinterpret_cast<const float *>(row) + chan);
#pragma unroll
        for (int i = 0; i < 4; ++i) r.v[i] = __ldg(q + i);
    }
}
template <bool BF16>
__device__ __forceinline__ float chan_of(const Raw16<BF16> &r, int c)      // c < 16, compile-time after unrolling
{
    if (BF16) {
        const uint4 &t = r.v[c >> 3];
        const int w = (c >> 1) & 3;
        const unsigned u = w == 0 ? t.x : w == 1 ? t.y : w == 2 ? t.z : t.w;
        return (c & 1) ? bf16hi_to_f32(u) : bf16lo_to_f32(u);
    } else {
        const uint4 &t = r.v[c >> 2];
        const int w = c & 3;
        return __uint_as_float(w == 0 ? t.x : w == 1 ? t.y : w == 2 ? t.z : t.w);
    }
}

// G: 32 (the warp's two spans are two groups), 64 (one group), 128 (half a group; NW = 2 warps share a group)
template <int BITS, int G, bool BF16, bool M16>
__global__ void __launch_bounds__(LR_THREADS, LR_CTAS_PER_SM) quant_keys_lowrank_kernel(const LrParams p)
{
    constexpr float L = float((1 << BITS) - 1);
    constexpr int NW = G == 128 ? 2 : 1;
    constexpr int SPG = G / 32;                     // spans per group
    constexpr int PER_ACC = 16 / BITS;              // codes accumulated exactly in one float
    constexpr int WORDS_PER_BLK = BLK * BITS / 32;
    constexpr bool TWO_GROUPS = G == 32;

    __shared__ __align__(16) float table[D * ROW];
    __shared__ float2 meta_all[LR_WARPS][2][BLK];   // (scale, zero) of the block just swept, per warp and span
    __shared__ float2 red_all[LR_WARPS / 2][2][2];  // G = 128: [team][parity][warp of the team] (min, max)

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int team = warp / NW, wteam = warp % NW;
    const int head = blockIdx.y;
    {
        const float4 *src = reinterpret_cast<const float4 *>(p.table + (long long)head * D * ROW);
        for (int i = threadIdx.x; i < D * ROW / 4; i += LR_THREADS)
            if (SQ_CHK_G(p.status, src + i, 16, p.x_table)) reinterpret_cast<float4 *>(table)[i] = __ldg(src + i);
    }
    __syncthreads();
    float2(*meta)[BLK] = meta_all[warp];

    constexpr int TEAMS = LR_WARPS / NW;
    for (int tt = blockIdx.x * TEAMS + team; tt < p.team_tasks; tt += gridDim.x * TEAMS) {
        // the two 32-token spans of this warp
        const void *row[2];
        unsigned char *cptr[2];
        long long meta_off[2];
        bool active[2];
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            int span = (tt * NW + wteam) * 2 + s;
            active[s] = span < p.spans_per_head;
            if (!active[s]) span = p.spans_per_head - 1;            // an odd count: the spare span redoes the last one, stores nothing
            const int group = span / SPG, sub = span % SPG;
            const int b = group / p.groups_per_bh, grp = group - b * p.groups_per_bh;
            const int tok = grp * G + sub * 32 + lane;
            const long long out_tok0 = (long long)b * p.osb + (long long)head * p.osh;
            cptr[s] = p.codes + (out_tok0 + tok) * (D * BITS / 8);
            meta_off[s] = (out_tok0 / G + grp) * D + lane;
            const long long off = (long long)b * p.sb + (long long)head * p.sh + (long long)tok * p.st;
            row[s] = BF16 ? static_cast<const void *>(reinterpret_cast<const __nv_bfloat16 *>(p.k) + off)
                          : static_cast<const void *>(reinterpret_cast<const float *>(p.k) + off);
        }
        u64 sp[2][R / 2];                                           // the tokens' states, packed in pairs
#pragma unroll
        for (int s = 0; s < 2; ++s)
#pragma unroll
            for (int i = 0; i < R / 2; ++i) sp[s][i] = 0ull;

#pragma unroll 1
        for (int blk = 0; blk < NBLK; ++blk) {
            Raw16<BF16> raw[2];
            float cacc[2][BLK / PER_ACC];
            const float *tab = table + blk * BLK * ROW;
#pragma unroll
            for (int jj = 0; jj < BLK; ++jj) {
                if (jj % 16 == 0) {
#pragma unroll
                    for (int s = 0; s < 2; ++s)
                        if (SQ_CHK_G(p.status, static_cast<const char *>(row[s]) + (blk * BLK + jj) * (BF16 ? 2 : 4), 16 * (BF16 ? 2 : 4), p.x_k))
                            load16<BF16>(raw[s], row[s], blk * BLK + jj);
                }
                const ulonglong2 v01 = *reinterpret_cast<const ulonglong2 *>(tab + jj * ROW);
                const ulonglong2 v23 = *reinterpret_cast<const ulonglong2 *>(tab + jj * ROW + 4);
                float x[2], m[2], Mx[2];
#pragma unroll
                for (int s = 0; s < 2; ++s) {                       // x_j = k_j + v_j . s
                    u64 acc = pack2(chan_of<BF16>(raw[s], jj % 16), 0.0f);
                    acc = ffma2(v01.x, sp[s][0], acc);
                    acc = ffma2(v01.y, sp[s][1], acc);
                    acc = ffma2(v23.x, sp[s][2], acc);
                    acc = ffma2(v23.y, sp[s][3], acc);
                    x[s] = __fadd_rn(lo_of(acc), hi_of(acc));
                }
                if (TWO_GROUPS) {
#pragma unroll
                    for (int s = 0; s < 2; ++s) { m[s] = warp_min(x[s]); Mx[s] = warp_max(x[s]); }
                } else {
                    float mm = warp_min(min_nan(x[0], x[1])), MM = warp_max(max_nan(x[0], x[1]));
                    if (NW > 1) {
                        float2 *slot = red_all[team][jj & 1];
                        if (lane == 0) slot[wteam] = make_float2(mm, MM);
                        asm volatile("bar.sync %0, %1;" ::"r"(1 + team), "r"(32 * NW) : "memory");
                        const float2 o = slot[wteam ^ 1];
                        mm = min_nan(mm, o.x);
                        MM = max_nan(MM, o.y);
                    }
                    m[0] = m[1] = mm;
                    Mx[0] = Mx[1] = MM;
                }
                const ulonglong2 c01 = *reinterpret_cast<const ulonglong2 *>(tab + jj * ROW + R);
                const ulonglong2 c23 = *reinterpret_cast<const ulonglong2 *>(tab + jj * ROW + R + 4);
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    const float rng = __fsub_rn(Mx[s], m[s]);
                    // the correctly rounded quotient where the decision is exact (channel 0, the only uncorrected one);
                    // elsewhere rng * RN(1 / L), one instruction, within an ulp of it (as in the dense kernel)
                    float scale = (jj == 0 && blk == 0) ? div_by_levels<BITS>(rng) : __fmul_rn(rng, 1.0f / L), zero = m[s];
                    float rcp, y0, dlt;
                    if (M16) {
                        scale = __half2float(__float2half_rn(scale));
                        zero = __half2float(__float2half_rn(zero));
                        dlt = __fsub_rn(x[s], zero);
                        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(rcp) : "f"(scale));
                        rcp = scale > 0.0f ? rcp : 0.0f;
                        y0 = __fmaf_rn(dlt, rcp, kMagic);
                    } else {
                        dlt = __fsub_rn(x[s], zero);
                        const float dltL = __fmul_rn(dlt, L);
                        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(rcp) : "f"(fmaxf(rng, 1e-30f)));
                        y0 = __fmaf_rn(dltL, rcp, kMagic);
                    }
                    float c = __fsub_rn(y0, kMagic);
                    float e = __fmaf_rn(c, scale, -dlt);
                    if (jj == 0 && blk == 0) {
                        // channel 0 is a raw input, where exact ties are structural: settle the rounding through the exact
                        // remainder, ties to the even code (see sweep_block in keys.cu)
                        const float thr = __uint_as_float(__float_as_uint(0.5f * scale) - (__float_as_uint(y0) & 1u));
                        const float adj = (e > thr) ? -1.0f : ((e < -thr) ? 1.0f : 0.0f);
                        c = __fadd_rn(c, adj);
                        e = __fmaf_rn(adj, scale, e);
                    }
                    if (M16) {
                        const float cc = fminf(fmaxf(c, 0.0f), L);
                        e = cc == c ? e : __fmaf_rn(cc, scale, -dlt);
                        c = cc;
                    }
                    if (jj % PER_ACC == 0) cacc[s][jj / PER_ACC] = c;
                    else cacc[s][jj / PER_ACC] = __fmaf_rn(c, float(1 << ((jj % PER_ACC) * BITS)), cacc[s][jj / PER_ACC]);
                    if (lane == 0 && (TWO_GROUPS || s == 0)) meta[s][jj] = make_float2(scale, zero);
                    const u64 ee = pack2(e, e);                     // s += e_j c_j
                    sp[s][0] = ffma2(ee, c01.x, sp[s][0]);
                    sp[s][1] = ffma2(ee, c01.y, sp[s][1]);
                    sp[s][2] = ffma2(ee, c23.x, sp[s][2]);
                    sp[s][3] = ffma2(ee, c23.y, sp[s][3]);
                }
            }
            __syncwarp();
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                if (!active[s]) continue;
                uint32_t cw[WORDS_PER_BLK];
#pragma unroll
                for (int w = 0; w < WORDS_PER_BLK; ++w)
                    cw[w] = (uint32_t)__float2int_rn(cacc[s][2 * w]) | ((uint32_t)__float2int_rn(cacc[s][2 * w + 1]) << 16);
                unsigned char *cp = cptr[s] + blk * (BLK * BITS / 8);
                if (!SQ_CHK_G(p.status, cp, BLK * BITS / 8, p.x_codes)) {
                } else if (WORDS_PER_BLK == 2)
                    *reinterpret_cast<uint2 *>(cp) = make_uint2(cw[0], cw[1]);
                else
                    *reinterpret_cast<uint4 *>(cp) = make_uint4(cw[0], cw[1], cw[WORDS_PER_BLK > 2 ? 2 : 0], cw[WORDS_PER_BLK > 2 ? 3 : 0]);
                // the group's metadata: one store per group (span 0 of warp 0 of the team unless the spans are groups)
                if ((TWO_GROUPS || (s == 0 && wteam == 0)) &&
                    SQ_CHK_G(p.status, static_cast<char *>(p.scales) + (meta_off[s] + blk * BLK) * (M16 ? 2 : 4), M16 ? 2 : 4, p.x_scales) &&
                    SQ_CHK_G(p.status, static_cast<char *>(p.zeros) + (meta_off[s] + blk * BLK) * (M16 ? 2 : 4), M16 ? 2 : 4, p.x_zeros)) {
                    const float2 sz = meta[s][lane];                 // lane = channel within the block
                    if (M16) {
                        reinterpret_cast<__half *>(p.scales)[meta_off[s] + blk * BLK] = __float2half_rn(sz.x);   // exact
                        reinterpret_cast<__half *>(p.zeros)[meta_off[s] + blk * BLK] = __float2half_rn(sz.y);
                    } else {
                        reinterpret_cast<float *>(p.scales)[meta_off[s] + blk * BLK] = sz.x;
                        reinterpret_cast<float *>(p.zeros)[meta_off[s] + blk * BLK] = sz.y;
                    }
                    if (!(sz.x > 0.0f && sz.x < __int_as_float(0x7f800000)))
                        atomicOr(p.status, sz.x == 0.0f ? SQUAT_FLAG_ZERO_RANGE : SQUAT_FLAG_NONFINITE);
                }
            }
            __syncwarp();                                           // meta is rewritten by the next block's sweep
        }
    }
}

template <int BITS, int G>
int launch_lowrank(const LrParams &p, int H, int dtype, int meta16, cudaStream_t st)
{
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    constexpr int TEAMS = LR_WARPS / (G == 128 ? 2 : 1);
    const int ctas_needed = (p.team_tasks + TEAMS - 1) / TEAMS;
    int per_head = (2 * LR_CTAS_PER_SM * sms + H - 1) / H;   // two waves of the resident CTAs, over all heads
    if (per_head > ctas_needed) per_head = ctas_needed;
    if (per_head < 1) per_head = 1;
    const dim3 grid(per_head, H);
#define SQ_LR(BF, MM) quant_keys_lowrank_kernel<BITS, G, BF, MM><<<grid, LR_THREADS, 0, st>>>(p)
    if (dtype == SQUAT_BF16) { if (meta16) SQ_LR(true, true); else SQ_LR(true, false); }
    else { if (meta16) SQ_LR(false, true); else SQ_LR(false, false); }
#undef SQ_LR
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return SQUAT_OK;
}

}  // namespace

int squat_launch_lowrank_tables(squat_subspace *s, int rank_r, double lambda, cudaStream_t st)
{
    lowrank_table_kernel<<<s->n_kv_heads, D, 0, st>>>(s->eigval, s->eigvec, rank_r, lambda, s->lr_table);
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return SQUAT_OK;
}

int squat_launch_quant_keys_lowrank(const float *table, const void *k, int dtype, int batch, int H, int T,
                                    long long sb, long long sh, long long st_, int bits, int G,
                                    unsigned char *codes, void *scales, void *zeros,
                                    long long osb, long long osh, unsigned *status, int meta16, cudaStream_t st)
{
    LrParams p;
    p.table = table; p.k = k; p.sb = sb; p.sh = sh; p.st = st_;
    p.codes = codes; p.scales = scales; p.zeros = zeros; p.osb = osb; p.osh = osh;
    p.groups_per_bh = T / G;
    const long long spans = (long long)batch * T / 32;
    if (spans == 0) return SQUAT_OK;
    if (spans > 0x3fffffffLL) return SQUAT_ERR_UNSUPPORTED;          // spans are counted in 32 bits
    p.spans_per_head = (int)spans;
    const int spans_per_task = G == 128 ? 4 : 2;
    p.team_tasks = (int)((spans + spans_per_task - 1) / spans_per_task);
    p.status = status;
#ifdef SQUAT_CHECKED
    {
        const unsigned long long es = dtype == SQUAT_BF16 ? 2 : 4, ms = meta16 ? 2 : 4;
        p.x_k = {k, (unsigned long long)((batch - 1) * sb + (H - 1) * sh + (long long)(T - 1) * st_ + D) * es};
        p.x_codes = {codes, (unsigned long long)((batch - 1) * osb + (H - 1) * osh + T) * (D * bits / 8)};
        const unsigned long long meta_elems = (unsigned long long)(((batch - 1) * osb + (H - 1) * osh) / G + T / G) * D;
        p.x_scales = {scales, meta_elems * ms};
        p.x_zeros = {zeros, meta_elems * ms};
        p.x_table = {table, (unsigned long long)H * D * ROW * 4};
    }
#endif
    if (bits == 2) {
        if (G == 32) return launch_lowrank<2, 32>(p, H, dtype, meta16, st);
        if (G == 64) return launch_lowrank<2, 64>(p, H, dtype, meta16, st);
        if (G == 128) return launch_lowrank<2, 128>(p, H, dtype, meta16, st);
    } else if (bits == 4) {
        if (G == 32) return launch_lowrank<4, 32>(p, H, dtype, meta16, st);
        if (G == 64) return launch_lowrank<4, 64>(p, H, dtype, meta16, st);
        if (G == 128) return launch_lowrank<4, 128>(p, H, dtype, meta16, st);
    }
    return SQUAT_ERR_UNSUPPORTED;
}
