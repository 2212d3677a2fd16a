// Key quantization with error feedback: Algorithm 1, function Quant, with the update of
// Eq. (3) / Eq. (update_block) applied through the assembled matrix W (W[j'][j] multiplies the
// rounding error of channel j into channel j' > j), and the quantizer of Section 2.
//
// Mapping.  A group is G consecutive tokens of one (batch, head); its channels must be visited in
// order, and each channel's grid needs min/max over the group's tokens.  So: lane = token, one warp
// (G = 32) or a team of G/32 warps per group, and the token's whole 128-channel working row lives
// in that lane's registers as 64 packed float pairs.  Channel j:
//     m, M   = warp min / max (redux.sync on f32)              -> scale = (M-m)/L, zero = m
//     c      = clamp(rint((x_j - m)/scale))                     (binary32 sequence, see values.cu)
//     e      = fma(c, scale, -(x_j - m))                        (= deq(qtz(x_j)) - x_j)
//     x_j'  += e * W[j'][j]  for j' > j                          packed fma.rn.f32x2, W row j is a
//                                                               shared-memory broadcast (LDS.128)
// The loop over j is fully unrolled so every register index is static.  The d x d matrix of the
// CTA's current head sits in shared memory (64 KB, stored transposed: row j = update vector of j).
// CTAs are persistent: each takes a contiguous range of groups ordered head-major, so W is
// reloaded only when the range crosses a head.
//
// Work per key vector: 8128 fp32 FMA (dense triangle, g = 1) -> bound by the FP32 pipes, not HBM.
#include "squat_internal.cuh"

namespace {

constexpr int D = SQUAT_D;
constexpr int NPAIR = D / 2;
constexpr float kMagic = 12582912.0f;
constexpr float kTieBand = 0.5f - 1e-5f;
constexpr int KEY_THREADS = 384;

typedef unsigned long long u64;

__device__ __forceinline__ u64 pack2(float lo, float hi)
{
    u64 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ float lo_of(u64 v)
{
    float lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
    return lo;
}
__device__ __forceinline__ float hi_of(u64 v)
{
    float lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
    return hi;
}
__device__ __forceinline__ u64 ffma2(u64 a, u64 b, u64 c)
{
    u64 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ float warp_min(float x)
{
    float r;
    asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ float warp_max(float x)
{
    float r;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ void team_barrier(int id, int nthreads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// Correctly rounded  rng / L  for L = 3 or 15 (q' = q + (rng - L q) * RN(1/L); checked against
// true division over full mantissa ranges on the host).
template <int BITS>
__device__ __forceinline__ float div_by_levels(float rng)
{
    constexpr float L = float((1 << BITS) - 1);
    constexpr float invL = 1.0f / L;
    const float q = __fmul_rn(rng, invL);
    const float r = __fmaf_rn(-L, q, rng);
    return __fmaf_rn(r, invL, q);
}

// Slow path for an element within 1e-5 of a rounding midpoint: the exact binary32 sequence.
template <int BITS>
__device__ __noinline__ float exact_code(float dlt, float scale)
{
    constexpr float L = float((1 << BITS) - 1);
    return fminf(fmaxf(rintf(__fdiv_rn(dlt, scale)), 0.0f), L);
}

struct KeyParams {
    const float *Wt;          // [H, D, D] transposed update matrices
    const void *k;
    long long sb, sh, st;     // element strides of k
    unsigned char *codes;
    float *scales, *zeros;
    long long osb, osh;       // output strides in tokens
    int B, H, T;
    int groups_per_bh;        // T / G
    long long total_groups;   // H * B * groups_per_bh, ordered (h, b, grp)
    unsigned *status;
};

template <int BITS, int NW, bool BF16>
__global__ void __launch_bounds__(KEY_THREADS, 1) quant_keys_kernel(const KeyParams p)
{
    constexpr float L = float((1 << BITS) - 1);
    constexpr int G = 32 * NW;
    constexpr int NTEAMS = KEY_THREADS / 32 / NW;
    constexpr int NWORDS = D * BITS / 32;
    constexpr int PER_WORD = 32 / BITS;
    extern __shared__ __align__(16) float smem[];
    float *Ws = smem;                                    // [D][D]
    float2 *red = reinterpret_cast<float2 *>(smem + D * D);   // [NTEAMS][2][NW] (min, max)

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int team = warp / NW;
    const int wteam = warp % NW;

    const long long lo = p.total_groups * blockIdx.x / gridDim.x;
    const long long hi = p.total_groups * (blockIdx.x + 1) / gridDim.x;
    const long long groups_per_head = (long long)p.B * p.groups_per_bh;

    long long pos = lo;
    while (pos < hi) {
        const int h = (int)(pos / groups_per_head);
        long long seg_end = (long long)(h + 1) * groups_per_head;
        if (seg_end > hi) seg_end = hi;

        __syncthreads();                                 // everyone is done with the previous head's W
        {
            const float4 *src = reinterpret_cast<const float4 *>(p.Wt + (long long)h * D * D);
            float4 *dst = reinterpret_cast<float4 *>(Ws);
            for (int i = threadIdx.x; i < D * D / 4; i += KEY_THREADS) dst[i] = __ldg(src + i);
        }
        __syncthreads();

        for (long long gi = pos + team; gi < seg_end; gi += NTEAMS) {
            const long long in_head = gi - (long long)h * groups_per_head;
            const int b = (int)(in_head / p.groups_per_bh);
            const int grp = (int)(in_head % p.groups_per_bh);
            const int tok = grp * G + wteam * 32 + lane;

            // ---- load this lane's token row into registers --------------------------------
            u64 xp[NPAIR];
            if (BF16) {
                const uint4 *src = reinterpret_cast<const uint4 *>(
                    reinterpret_cast<const __nv_bfloat16 *>(p.k) + (long long)b * p.sb + (long long)h * p.sh + (long long)tok * p.st);
#pragma unroll
                for (int i = 0; i < D / 8; ++i) {
                    const uint4 r = ldg128(src + i);
                    xp[4 * i + 0] = pack2(bf16lo_to_f32(r.x), bf16hi_to_f32(r.x));
                    xp[4 * i + 1] = pack2(bf16lo_to_f32(r.y), bf16hi_to_f32(r.y));
                    xp[4 * i + 2] = pack2(bf16lo_to_f32(r.z), bf16hi_to_f32(r.z));
                    xp[4 * i + 3] = pack2(bf16lo_to_f32(r.w), bf16hi_to_f32(r.w));
                }
            } else {
                const uint4 *src = reinterpret_cast<const uint4 *>(
                    reinterpret_cast<const float *>(p.k) + (long long)b * p.sb + (long long)h * p.sh + (long long)tok * p.st);
#pragma unroll
                for (int i = 0; i < D / 4; ++i) {
                    const uint4 r = ldg128(src + i);
                    xp[2 * i + 0] = pack2(__uint_as_float(r.x), __uint_as_float(r.y));
                    xp[2 * i + 1] = pack2(__uint_as_float(r.z), __uint_as_float(r.w));
                }
            }

            const long long out_tok0 = (long long)b * p.osb + (long long)h * p.osh;   // token offset of (b, h)
            float *sc_out = p.scales + (out_tok0 / G + grp) * D;
            float *zr_out = p.zeros + (out_tok0 / G + grp) * D;
            uint32_t cw[NWORDS];
            float my_scale = 0.0f, my_zero = 0.0f;
            unsigned flags = 0;

            // ---- the sequential sweep over channels ---------------------------------------
#pragma unroll
            for (int j = 0; j < D; ++j) {
                const float xj = (j & 1) ? hi_of(xp[j >> 1]) : lo_of(xp[j >> 1]);
                float m = warp_min(xj);
                float Mx = warp_max(xj);
                if (NW > 1) {
                    float2 *slot = red + (team * 2 + (j & 1)) * NW;
                    if (lane == 0) slot[wteam] = make_float2(m, Mx);
                    team_barrier(1 + team, 32 * NW);
#pragma unroll
                    for (int w = 0; w < NW; ++w) {
                        const float2 o = slot[w];
                        m = fminf(m, o.x);
                        Mx = fmaxf(Mx, o.y);
                    }
                }
                const float scale = div_by_levels<BITS>(__fsub_rn(Mx, m));
                const bool ok = scale > 0.0f && scale < __int_as_float(0x7f800000);
                if (!ok) flags |= (scale == 0.0f) ? SQUAT_FLAG_ZERO_RANGE : SQUAT_FLAG_NONFINITE;
                const float rcp = ok ? __frcp_rn(scale) : 0.0f;
                const float dlt = __fsub_rn(xj, m);
                const float y = __fmaf_rn(dlt, rcp, kMagic);
                float c = __fsub_rn(y, kMagic);
                const float res = __fmaf_rn(dlt, rcp, -c);
                if (__any_sync(0xffffffffu, fabsf(res) >= kTieBand) && ok) {
                    if (fabsf(res) >= kTieBand) c = exact_code<BITS>(dlt, scale);
                }
                const float e = __fmaf_rn(c, scale, -dlt);
                const u64 ee = pack2(e, e);

                // push the error onto the later channels:  x[j'] += e * W[j'][j]
                const float *wrow = Ws + j * D;
#pragma unroll
                for (int q = (j + 1) / 4; q < D / 4; ++q) {
                    const ulonglong2 w = *reinterpret_cast<const ulonglong2 *>(wrow + 4 * q);
                    if (2 * q >= (j + 1) / 2) xp[2 * q] = ffma2(ee, w.x, xp[2 * q]);
                    xp[2 * q + 1] = ffma2(ee, w.y, xp[2 * q + 1]);
                }

                // bookkeeping: code bits, and the (scale, zero) of channel j parked in lane j % 32
                const uint32_t cbits = (uint32_t)(int)c;
                if (j % PER_WORD == 0) cw[j / PER_WORD] = cbits;
                else cw[j / PER_WORD] |= cbits << ((j % PER_WORD) * BITS);
                if (lane == (j & 31)) { my_scale = scale; my_zero = m; }
                if ((j & 31) == 31 && wteam == 0) {
                    sc_out[(j & ~31) + lane] = my_scale;
                    zr_out[(j & ~31) + lane] = my_zero;
                }
            }

            // ---- write this token's packed codes -------------------------------------------
            uint4 *cp = reinterpret_cast<uint4 *>(p.codes + (out_tok0 + tok) * (D * BITS / 8));
#pragma unroll
            for (int i = 0; i < NWORDS / 4; ++i) cp[i] = make_uint4(cw[4 * i], cw[4 * i + 1], cw[4 * i + 2], cw[4 * i + 3]);
            if (flags) atomicOr(p.status, flags);
        }
        pos = seg_end;
    }
}

template <int BITS, int NW>
int launch_keys(const KeyParams &p, int dtype, cudaStream_t st)
{
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    constexpr int NTEAMS = KEY_THREADS / 32 / NW;
    const size_t smem = sizeof(float) * D * D + sizeof(float2) * NTEAMS * 2 * NW;
    long long want = (p.total_groups + NTEAMS - 1) / NTEAMS;
    const int grid = (int)(want < sms ? want : sms);
    if (dtype == SQUAT_BF16) {
        SQUAT_CUDA(cudaFuncSetAttribute(quant_keys_kernel<BITS, NW, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        quant_keys_kernel<BITS, NW, true><<<grid, KEY_THREADS, smem, st>>>(p);
    } else {
        SQUAT_CUDA(cudaFuncSetAttribute(quant_keys_kernel<BITS, NW, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        quant_keys_kernel<BITS, NW, false><<<grid, KEY_THREADS, smem, st>>>(p);
    }
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return SQUAT_OK;
}

}  // namespace

int squat_launch_quant_keys(const float *Wt, const void *k, int dtype, int batch, int H, int T,
                            long long sb, long long sh, long long st_, int bits, int G,
                            unsigned char *codes, float *scales, float *zeros,
                            long long osb, long long osh, unsigned *status, cudaStream_t st)
{
    KeyParams p;
    p.Wt = Wt; p.k = k; p.sb = sb; p.sh = sh; p.st = st_;
    p.codes = codes; p.scales = scales; p.zeros = zeros; p.osb = osb; p.osh = osh;
    p.B = batch; p.H = H; p.T = T; p.groups_per_bh = T / G;
    p.total_groups = (long long)H * batch * (T / G);
    p.status = status;
    if (p.total_groups == 0) return SQUAT_OK;
    if (bits == 2) {
        if (G == 32) return launch_keys<2, 1>(p, dtype, st);
        if (G == 64) return launch_keys<2, 2>(p, dtype, st);
        if (G == 128) return launch_keys<2, 4>(p, dtype, st);
    } else if (bits == 4) {
        if (G == 32) return launch_keys<4, 1>(p, dtype, st);
        if (G == 64) return launch_keys<4, 2>(p, dtype, st);
        if (G == 128) return launch_keys<4, 4>(p, dtype, st);
    }
    return SQUAT_ERR_UNSUPPORTED;
}
