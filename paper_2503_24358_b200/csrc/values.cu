// Per-token value quantization (Section 2 "Quantization"; Appendix C: d channels of a token in
// d/G groups of G) and dequantization (deq(c) = c * Delta + m) for both cache layouts.
//
// HBM-bound streaming kernels.  One thread owns one (token, channel-group): it reads its G
// consecutive channels with 128-bit loads (consecutive lanes read consecutive 16*G/8-byte
// pieces, so a warp covers a contiguous span), reduces min/max in registers, and writes
// G*b/8 code bytes plus one scale and one zero -- all contiguous across the warp.
//
// The rounding decision is the IEEE binary32 sequence  Delta = (M-m)/L, t = (x-m)/Delta,
// c = clamp(rint(t), 0, L).  The fast path multiplies by RN(1/Delta) and rounds once; it can
// differ from the sequence above only when t is within ~1e-6 of a half-integer, so any
// element within 1e-5 of one is redone with a correctly rounded division.
//
// M16 instances store scale and zero-point as IEEE binary16 (the 18.75 % cache of the paper's "KV size" columns):
// Delta = half(Delta32), z = half(m), and the decision t = (x - z) / Delta is taken against those stored values,
// so codes are clamped (a rounded zero-point can lie above the minimum).
#include "squat_internal.cuh"
#include <cuda_fp16.h>

namespace {

constexpr float kMagic = 12582912.0f;   // 1.5 * 2^23: adding it rounds to an integer (ties to even)
constexpr float kTieBand = 0.5f - 1e-5f;

typedef unsigned long long u64;
__device__ __forceinline__ u64 pk2(float lo, float hi) { u64 r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi)); return r; }
__device__ __forceinline__ void unpk2(u64 v, float &lo, float &hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ u64 sub2(u64 a, u64 b) { u64 d; asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d; }
__device__ __forceinline__ u64 fma2(u64 a, u64 b, u64 c) { u64 d; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c)); return d; }

// NaN-propagating min / max: a NaN input makes the group's scale NaN, which is reported (SQUAT_FLAG_NONFINITE) and gives
// codes 0, instead of being dropped by the reduction.
__device__ __forceinline__ float min_nan(float a, float b) { float r; asm("min.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b)); return r; }
__device__ __forceinline__ float max_nan(float a, float b) { float r; asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b)); return r; }

// Exact binary32 decision for one element next to a rounding midpoint (rare; kept out of line).
template <int BITS>
__device__ __noinline__ uint32_t exact_code_bits(float dlt, float delta)
{
    constexpr float L = float((1 << BITS) - 1);
    return (uint32_t)(int)fminf(fmaxf(rintf(__fdiv_rn(dlt, delta)), 0.0f), L);
}

template <int G, bool BF16>
struct ValRaw {
    static constexpr int NV = BF16 ? G / 8 : G / 4;      // 128-bit pieces of one group
    uint4 v[NV];
    __device__ __forceinline__ float get(int i) const     // channel i of the group, exact widening
    {
        if (BF16) {
            const uint4 &r = v[i / 8];
            const uint32_t w = (i % 8) / 2 == 0 ? r.x : (i % 8) / 2 == 1 ? r.y : (i % 8) / 2 == 2 ? r.z : r.w;
            return (i & 1) ? bf16hi_to_f32(w) : bf16lo_to_f32(w);
        } else {
            const uint4 &r = v[i / 4];
            const uint32_t w = i % 4 == 0 ? r.x : i % 4 == 1 ? r.y : i % 4 == 2 ? r.z : r.w;
            return __uint_as_float(w);
        }
    }
};

template <int G, int BITS, bool BF16, bool M16>
__global__ void __launch_bounds__(256) quant_values_kernel(
    const void *__restrict__ v, long long n_units, int H, int T, int ng,
    long long sb, long long sh, long long st, unsigned char *__restrict__ codes,
    void *__restrict__ scales, void *__restrict__ zeros, long long osb, long long osh,
    int row_bytes, unsigned *__restrict__ status)
{
    constexpr float L = float((1 << BITS) - 1);
    constexpr int PER_WORD = 32 / BITS;
    constexpr int NWORDS = G / PER_WORD;
    using Raw = ValRaw<G, BF16>;
    constexpr bool PREFETCH = false;              // keep the next unit's data in flight while this one computes
    const long long stride = (long long)gridDim.x * blockDim.x;

    auto in_ptr = [&](long long u) -> const uint4 * {
        const int q = (int)(u % ng);
        const long long tok = u / ng;
        const int t = (int)(tok % T);
        const long long bh = tok / T;
        const long long off = (bh / H) * sb + (bh % H) * sh + (long long)t * st + (long long)q * G;
        return BF16 ? reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(v) + off)
                    : reinterpret_cast<const uint4 *>(reinterpret_cast<const float *>(v) + off);
    };
    auto load = [&](Raw &r, long long u) {
        const uint4 *p = in_ptr(u);
#pragma unroll
        for (int i = 0; i < Raw::NV; ++i) r.v[i] = ldg128(p + i);
    };

    long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    Raw nxt;
    if (PREFETCH && u < n_units) load(nxt, u);
    for (; u < n_units; u += stride) {
        Raw raw;
        if (PREFETCH) {
            raw = nxt;
            if (u + stride < n_units) load(nxt, u + stride);
        } else {
            load(raw, u);
        }
        const int q = (int)(u % ng);
        const long long tok = u / ng;
        const int t = (int)(tok % T);
        const long long bh = tok / T;
        const long long out_tok = (bh / H) * osb + (bh % H) * osh + t;

        float m, Mx;
        if (BF16) {
            // min / max on packed bf16 pairs (exact), then across the pair
            __nv_bfloat162 mn2, mx2;
#pragma unroll
            for (int i = 0; i < Raw::NV; ++i) {
                const uint32_t w[4] = {raw.v[i].x, raw.v[i].y, raw.v[i].z, raw.v[i].w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const __nv_bfloat162 pr = *reinterpret_cast<const __nv_bfloat162 *>(&w[k]);
                    if (i == 0 && k == 0) { mn2 = pr; mx2 = pr; }
                    else { mn2 = __hmin2_nan(mn2, pr); mx2 = __hmax2_nan(mx2, pr); }
                }
            }
            m = min_nan(__low2float(mn2), __high2float(mn2));
            Mx = max_nan(__low2float(mx2), __high2float(mx2));
        } else {
            m = raw.get(0); Mx = m;
#pragma unroll
            for (int i = 1; i < G; ++i) { m = min_nan(m, raw.get(i)); Mx = max_nan(Mx, raw.get(i)); }
        }

        float delta = __fdiv_rn(__fsub_rn(Mx, m), L);
        if (M16) {                                         // the stored binary16 values decide
            delta = __half2float(__float2half_rn(delta));
            m = __half2float(__float2half_rn(m));
        }
        const bool ok = delta > 0.0f && delta < __int_as_float(0x7f800000);
        const float rcp = ok ? __frcp_rn(delta) : 0.0f;
        if (!ok) atomicOr(status, delta == 0.0f ? SQUAT_FLAG_ZERO_RANGE : SQUAT_FLAG_NONFINITE);

        // two channels per instruction (packed f32x2): dlt = x - m, y = dlt * rcp + magic, c = y - magic,
        // res = dlt * rcp - c; each half is the same IEEE operation as its scalar form
        const u64 m2 = pk2(m, m), rcp2 = pk2(rcp, rcp), magic2 = pk2(kMagic, kMagic);
        const uint32_t cmask = ok ? ((1u << BITS) - 1u) : 0u;       // no grid (constant or non-finite group): codes 0
        uint32_t words[NWORDS];
#pragma unroll
        for (int wd = 0; wd < NWORDS; ++wd) {
            uint32_t acc = 0;
#pragma unroll
            for (int k = 0; k < PER_WORD; k += 2) {
                const int i = wd * PER_WORD + k;
                const u64 dlt2 = sub2(pk2(raw.get(i), raw.get(i + 1)), m2);
                const u64 y2 = fma2(dlt2, rcp2, magic2);
                const u64 nc2 = sub2(magic2, y2);                       // -(y - magic), exact
                const u64 res2 = fma2(dlt2, rcp2, nc2);
                float ylo, yhi, rlo, rhi;
                unpk2(y2, ylo, yhi);
                unpk2(res2, rlo, rhi);
                if (M16) {                                  // rounded metadata: t may leave [0, L]
                    ylo = fminf(fmaxf(ylo, kMagic), kMagic + L);
                    yhi = fminf(fmaxf(yhi, kMagic), kMagic + L);
                }
                uint32_t cb0 = __float_as_uint(ylo) & cmask;
                uint32_t cb1 = __float_as_uint(yhi) & cmask;
                // next to a rounding midpoint (structural with coarse bf16 data): the exact sequence decides
                if (fmaxf(fabsf(rlo), fabsf(rhi)) >= kTieBand && ok) {
                    float dlo, dhi;
                    unpk2(dlt2, dlo, dhi);
                    if (fabsf(rlo) >= kTieBand) cb0 = exact_code_bits<BITS>(dlo, delta);
                    if (fabsf(rhi) >= kTieBand) cb1 = exact_code_bits<BITS>(dhi, delta);
                }
                acc |= (cb0 | (cb1 << BITS)) << (k * BITS);
            }
            words[wd] = acc;
        }

        unsigned char *cp = codes + out_tok * row_bytes + (long long)q * (G * BITS / 8);
        if (NWORDS % 4 == 0) {
#pragma unroll
            for (int i = 0; i < NWORDS / 4; ++i)
                reinterpret_cast<uint4 *>(cp)[i] = make_uint4(words[4 * i], words[4 * i + 1], words[4 * i + 2], words[4 * i + 3]);
        } else {
#pragma unroll
            for (int i = 0; i < NWORDS / 2; ++i)
                reinterpret_cast<uint2 *>(cp)[i] = make_uint2(words[2 * i], words[2 * i + 1]);
        }
        if (M16) {
            reinterpret_cast<__half *>(scales)[out_tok * ng + q] = __float2half_rn(delta);      // exact: already binary16 values
            reinterpret_cast<__half *>(zeros)[out_tok * ng + q] = __float2half_rn(m);
        } else {
            reinterpret_cast<float *>(scales)[out_tok * ng + q] = delta;
            reinterpret_cast<float *>(zeros)[out_tok * ng + q] = m;
        }
    }
}

// One thread dequantizes 16 consecutive channels of TOK = 4 or 8 consecutive tokens (same key group, so the 16
// scales and zeros are read once for all of them; 8 on large inputs, 4 where that would leave SMs without work).  Codes become floats through the 2^23 trick
// (exact), then one fma each: deq(c) = fma(c, scale, zero), rounded once.
template <int BITS, bool KEYS, bool OUT_BF16, bool M16, int TOK>
__global__ void __launch_bounds__(256, 4) dequant_kernel(
    const unsigned char *__restrict__ codes, const void *__restrict__ scales, const void *__restrict__ zeros,
    long long n_units, int H, int T, int d, int G, long long isb, long long ish, void *__restrict__ out)
{
    const int per_tok = d / 16;
    const int tq_per_row = (T + TOK - 1) / TOK;
    const int row_bytes = d * BITS / 8;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x; u < n_units; u += stride) {
        const int c16 = (int)(u % per_tok);
        const long long r = u / per_tok;
        const int t0 = (int)(r % tq_per_row) * TOK;
        const long long bh = r / tq_per_row;
        const int h = (int)(bh % H);
        const long long b = bh / H;
        const long long in_tok0 = b * isb + h * ish;
        float sc[16], zr[16];
        if (KEYS) {
            const long long base = (b * (isb / G) + h * (ish / G) + t0 / G) * d + c16 * 16;
            if (M16) {
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const uint4 s8 = __ldg(reinterpret_cast<const uint4 *>(reinterpret_cast<const __half *>(scales) + base) + i);
                    const uint4 z8 = __ldg(reinterpret_cast<const uint4 *>(reinterpret_cast<const __half *>(zeros) + base) + i);
                    const uint32_t sw[4] = {s8.x, s8.y, s8.z, s8.w}, zw[4] = {z8.x, z8.y, z8.z, z8.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const float2 sf = __half22float2(*reinterpret_cast<const __half2 *>(&sw[k]));
                        const float2 zf = __half22float2(*reinterpret_cast<const __half2 *>(&zw[k]));
                        sc[8 * i + 2 * k] = sf.x; sc[8 * i + 2 * k + 1] = sf.y;
                        zr[8 * i + 2 * k] = zf.x; zr[8 * i + 2 * k + 1] = zf.y;
                    }
                }
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float4 s4 = __ldg(reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(scales) + base) + i);
                    const float4 z4 = __ldg(reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(zeros) + base) + i);
                    sc[4 * i] = s4.x; sc[4 * i + 1] = s4.y; sc[4 * i + 2] = s4.z; sc[4 * i + 3] = s4.w;
                    zr[4 * i] = z4.x; zr[4 * i + 1] = z4.y; zr[4 * i + 2] = z4.z; zr[4 * i + 3] = z4.w;
                }
            }
        }
#pragma unroll
        for (int tt = 0; tt < TOK; ++tt) {
            const int t = t0 + tt;
            if (t >= T) break;
            const unsigned char *cp = codes + (in_tok0 + t) * row_bytes + c16 * (16 * BITS / 8);
            uint32_t w[2];
            if (BITS == 2) { w[0] = __ldg(reinterpret_cast<const uint32_t *>(cp)); w[1] = 0; }
            else { const uint2 rr = __ldg(reinterpret_cast<const uint2 *>(cp)); w[0] = rr.x; w[1] = rr.y; }
            float s1 = 0.0f, z1 = 0.0f;
            if (!KEYS) {
                const long long mi = (in_tok0 + t) * (d / G) + (c16 * 16) / G;
                if (M16) {
                    s1 = __half2float(__ldg(reinterpret_cast<const __half *>(scales) + mi));
                    z1 = __half2float(__ldg(reinterpret_cast<const __half *>(zeros) + mi));
                } else {
                    s1 = __ldg(reinterpret_cast<const float *>(scales) + mi);
                    z1 = __ldg(reinterpret_cast<const float *>(zeros) + mi);
                }
            }
            float y[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int bit = i * BITS;
                const uint32_t cb = (w[bit / 32] >> (bit % 32)) & ((1u << BITS) - 1u);
                const float c = __fsub_rn(__uint_as_float(0x4B000000u | cb), 8388608.0f);     // exact int -> float
                y[i] = KEYS ? __fmaf_rn(c, sc[i], zr[i]) : __fmaf_rn(c, s1, z1);
            }
            const long long o = ((bh * T) + t) * d + c16 * 16;
            if (OUT_BF16) {
                uint32_t pk[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    __nv_bfloat162 p2 = __floats2bfloat162_rn(y[2 * i], y[2 * i + 1]);
                    pk[i] = *reinterpret_cast<uint32_t *>(&p2);
                }
                uint4 *op = reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>(out) + o);
                op[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                op[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
            } else {
                float4 *op = reinterpret_cast<float4 *>(reinterpret_cast<float *>(out) + o);
#pragma unroll
                for (int i = 0; i < 4; ++i) op[i] = make_float4(y[4 * i], y[4 * i + 1], y[4 * i + 2], y[4 * i + 3]);
            }
        }
    }
}

int grid_for(long long n_threads, int block)
{
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    long long blocks = (n_threads + block - 1) / block;
    const long long cap = (long long)sms * 32;          // a multiple of the SM count; grid-stride covers the rest
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

template <int G, int BITS>
int launch_values(const void *v, int dtype, long long n_units, int H, int T, int ng, long long sb, long long sh,
                  long long st_, unsigned char *codes, void *scales, void *zeros, long long osb, long long osh,
                  int row_bytes, unsigned *status, int meta16, cudaStream_t st)
{
    const int grid = grid_for(n_units, 256);
#define SQ_VK(BF, MM) quant_values_kernel<G, BITS, BF, MM><<<grid, 256, 0, st>>>(v, n_units, H, T, ng, sb, sh, st_, codes, scales, zeros, osb, osh, row_bytes, status)
    if (dtype == SQUAT_BF16) { if (meta16) SQ_VK(true, true); else SQ_VK(true, false); }
    else { if (meta16) SQ_VK(false, true); else SQ_VK(false, false); }
#undef SQ_VK
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return SQUAT_OK;
}

}  // namespace

int squat_launch_quant_values(const void *v, int dtype, int batch, int H, int T, int d,
                              long long sb, long long sh, long long st_, int bits, int G,
                              unsigned char *codes, void *scales, void *zeros,
                              long long osb, long long osh, unsigned *status, int meta16, cudaStream_t st)
{
    const int ng = d / G;
    const long long n_units = (long long)batch * H * T * ng;
    if (n_units == 0) return SQUAT_OK;
    const int row_bytes = d * bits / 8;
#define SQ_V(GG, BB) return launch_values<GG, BB>(v, dtype, n_units, H, T, ng, sb, sh, st_, codes, scales, zeros, osb, osh, row_bytes, status, meta16, st)
    if (bits == 2) { if (G == 32) SQ_V(32, 2); if (G == 64) SQ_V(64, 2); if (G == 128) SQ_V(128, 2); }
    if (bits == 4) { if (G == 32) SQ_V(32, 4); if (G == 64) SQ_V(64, 4); if (G == 128) SQ_V(128, 4); }
#undef SQ_V
    return SQUAT_ERR_UNSUPPORTED;
}

int squat_launch_dequant(int kind, const unsigned char *codes, const void *scales, const void *zeros,
                         int batch, int H, int T, int d, int bits, int G, long long isb, long long ish,
                         void *out, int out_dtype, int meta16, cudaStream_t st)
{
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long long units8 = (long long)batch * H * ((T + 7) / 8) * (d / 16);       // threads with 8 tokens x 16 channels each
    const bool tok8 = units8 >= (long long)sms * 32 * 256;                           // enough of them to fill the grid cap
    const long long n_units = tok8 ? units8 : (long long)batch * H * ((T + 3) / 4) * (d / 16);
    if (n_units == 0) return SQUAT_OK;
    const int grid = grid_for(n_units, 256);
#define SQ_D1(BB, KK, OO, MM, TT) dequant_kernel<BB, KK, OO, MM, TT><<<grid, 256, 0, st>>>(codes, scales, zeros, n_units, H, T, d, G, isb, ish, out)
#define SQ_D(BB, KK, OO) do { if (meta16) { if (tok8) SQ_D1(BB, KK, OO, true, 8); else SQ_D1(BB, KK, OO, true, 4); } \
                              else { if (tok8) SQ_D1(BB, KK, OO, false, 8); else SQ_D1(BB, KK, OO, false, 4); } } while (0)
    const bool keys = kind == SQUAT_KEYS, obf = out_dtype == SQUAT_BF16;
    if (bits == 2) {
        if (keys) { if (obf) SQ_D(2, true, true); else SQ_D(2, true, false); }
        else { if (obf) SQ_D(2, false, true); else SQ_D(2, false, false); }
    } else if (bits == 4) {
        if (keys) { if (obf) SQ_D(4, true, true); else SQ_D(4, true, false); }
        else { if (obf) SQ_D(4, false, true); else SQ_D(4, false, false); }
    } else {
        return SQUAT_ERR_UNSUPPORTED;
    }
#undef SQ_D1
#undef SQ_D
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return SQUAT_OK;
}
