// Per-token value quantization (Section 2 "Quantization"; Appendix C: d channels of a token in
// d/G groups of G) and dequantization (deq(c) = c * Delta + m) for both cache layouts.
//
// HBM-bound streaming kernels, written to spend few instructions per element (the first version of the quantizer
// needed 15 per element and was bound by instruction issue at 70 % of the copy bandwidth).
//
// Quantizer.  A thread owns one 16-byte piece of the input (8 bf16 or 4 float32 channels), so a warp's load is one
// contiguous 512-byte span; the G channels of a group lie in G/8 (G/4) neighbouring lanes, which reduce min / max
// with warp shuffles.  The rounding decision is the IEEE binary32 sequence
//     Delta = (M - m) / L,   t = (x - m) / Delta,   c = clamp(rint(t), 0, L).
// Fast path: t is bracketed by  (x - m) * r (1 +- 2^-20)  with r the hardware reciprocal of Delta (1 ulp); both ends are
// rounded to integers by adding 1.5 * 2^23 (one fma each, ties to even).  rint is monotonic, so where the two ends
// agree that integer is rint(t); where they differ for any element of the piece (t within 1e-6 relative of a
// rounding midpoint -- structural with coarse bf16 data) the piece is redone with correctly rounded divisions.
// The codes are packed by integer shift-adds of the rounded floats' bit patterns (the constant upper bits are
// subtracted once).
//
// M16 instances store scale and zero-point as IEEE binary16 (the 18.75 % cache of the paper's "KV size" columns):
// Delta = half(Delta32), z = half(m), and the decision t = (x - z) / Delta is taken against those stored values,
// so codes are clamped (a rounded zero-point can lie above the minimum).
#include "squat_internal.cuh"
#include <cuda_fp16.h>

namespace {

constexpr float kMagic = 12582912.0f;   // 1.5 * 2^23: adding it rounds to an integer (ties to even)
constexpr unsigned kMagicBits = 0x4B400000u;

typedef unsigned long long u64;
__device__ __forceinline__ u64 pk2(float lo, float hi) { u64 r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi)); return r; }
__device__ __forceinline__ void unpk2(u64 v, float &lo, float &hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ u64 sub2(u64 a, u64 b) { u64 d; asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d; }
__device__ __forceinline__ u64 fma2(u64 a, u64 b, u64 c) { u64 d; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c)); return d; }

// NaN-propagating min / max: a NaN input makes the group's scale NaN, which is reported (SQUAT_FLAG_NONFINITE) and gives
// codes 0, instead of being dropped by the reduction.
__device__ __forceinline__ float min_nan(float a, float b) { float r; asm("min.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b)); return r; }
__device__ __forceinline__ float max_nan(float a, float b) { float r; asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b)); return r; }
__device__ __forceinline__ unsigned hmin2_nan_bits(unsigned a, unsigned b)
{
    const __nv_bfloat162 r = __hmin2_nan(*reinterpret_cast<const __nv_bfloat162 *>(&a), *reinterpret_cast<const __nv_bfloat162 *>(&b));
    return *reinterpret_cast<const unsigned *>(&r);
}
__device__ __forceinline__ unsigned hmax2_nan_bits(unsigned a, unsigned b)
{
    const __nv_bfloat162 r = __hmax2_nan(*reinterpret_cast<const __nv_bfloat162 *>(&a), *reinterpret_cast<const __nv_bfloat162 *>(&b));
    return *reinterpret_cast<const unsigned *>(&r);
}

// Correctly rounded  rng / L  for L = 3 or 15 and rng, rng / L in the normal range (q' = q + (rng - L q) * RN(1/L)).
template <int BITS>
__device__ __forceinline__ float div_by_levels(float rng)
{
    constexpr float L = float((1 << BITS) - 1);
    constexpr float invL = 1.0f / L;
    const float q = __fmul_rn(rng, invL);
    const float r = __fmaf_rn(-L, q, rng);
    return __fmaf_rn(r, invL, q);
}

// Exact binary32 decision for one element (rare; kept out of line).
template <int BITS>
__device__ __noinline__ uint32_t exact_code_bits(float dlt, float delta)
{
    constexpr float L = float((1 << BITS) - 1);
    return (uint32_t)(int)fminf(fmaxf(rintf(__fdiv_rn(dlt, delta)), 0.0f), L);
}

struct ValParams {
    const void *v;
    int H, T, ng;                         // ng = groups per token
    int ns, ns_shift;                     // ns = 32-channel spans per token (d / 32); its log2 when a power of two, else -1
    unsigned chunks_per_row;              // CTAs per (batch, head) row
    long long sb, sh, st;                 // element strides of v
    unsigned char *codes;
    void *scales, *zeros;
    long long osb, osh;                   // output strides in tokens
    int row_bytes;                        // code bytes per token
    unsigned *status;
#ifdef SQUAT_CHECKED
    SqExtent x_v, x_codes, x_scales, x_zeros;      // what the caller's tensors span
#endif
};

constexpr int VAL_THREADS = 256;

// The rare path of the quantizer, out of line so that the streaming code stays small.  `mask` has one bit set (at the
// element's bit position in the packed word) for every element of the word whose fast path could not decide; each is
// re-read from memory (it is in L1) and decided here, and its field of `word` replaced.  A scale outside the fast
// path's range (`fast` false, every element flagged): the exact sequence.  Else the element sits next to a rounding
// midpoint k + 1/2 (structural with coarse bf16 data): the sign of the exact remainder (x - m) - (k + 1/2) Delta (one
// fma: the product has at most 29 significant bits) says on which side the quotient lies; a zero remainder is an exact
// tie and goes to the even code; a remainder too small to be sure that the ROUNDED quotient is not the midpoint itself
// takes the correctly rounded division.
template <int BITS, bool BF16, bool M16>
__device__ __noinline__ unsigned patch_word(unsigned word, unsigned mask, const void *elems, float m, float delta, float ra,
                                            float rb, bool fast)
{
    constexpr float L = float((1 << BITS) - 1);
    while (mask) {
        const int pos = __ffs(mask) - 1, i = pos / BITS;
        mask &= mask - 1;
        const float x = BF16 ? __uint_as_float((unsigned)__ldg(reinterpret_cast<const unsigned short *>(elems) + i) << 16)
                             : __ldg(reinterpret_cast<const float *>(elems) + i);
        const float dl = __fsub_rn(x, m);
        float y;
        if (!fast) {
            y = kMagic + fminf(fmaxf(rintf(__fdiv_rn(dl, delta)), 0.0f), L);
        } else {
            const float ya = __fmaf_rn(dl, ra, kMagic), yb = __fmaf_rn(dl, rb, kMagic);
            y = ya;
            if (ya != yb) {
                const float lo = fminf(ya, yb), hi = fmaxf(ya, yb);
                const float kh = __fadd_rn(__fsub_rn(lo, kMagic), 0.5f);
                const float r = __fmaf_rn(-kh, delta, dl);
                if (r == 0.0f) y = (__float_as_uint(lo) & 1u) ? hi : lo;
                else if (fabsf(r) > fabsf(kh) * delta * 0x1p-21f) y = r > 0.0f ? hi : lo;
                else y = kMagic + fminf(fmaxf(rintf(__fdiv_rn(dl, delta)), 0.0f), L);
            }
            if (M16) y = fminf(fmaxf(y, kMagic), kMagic + L);
        }
        const unsigned field = ((1u << BITS) - 1u) << (BITS * i);
        word = (word & ~field) | ((__float_as_uint(y) << (BITS * i)) & field);
    }
    return word;
}

// One thread owns a span of 32 consecutive channels of one token in registers (4 or 8 16-byte loads in flight); a group
// of G channels is 1, 2 or 4 neighbouring lanes, which combine their min / max with warp shuffles.  One CTA works
// VAL_THREADS consecutive spans of one (batch, head) row -- grid (chunks of a row, heads, batch) -- so no index is divided
// out of a flat CTA number; a span's token is a shift (d / 32 a power of two) or one 32-bit division.
template <int G, int BITS, bool BF16, bool M16>
__global__ void __launch_bounds__(VAL_THREADS) quant_values_kernel(const ValParams p)
{
    constexpr float L = float((1 << BITS) - 1);
    constexpr int SPAN = 32;                        // channels per thread
    constexpr int LPG = G / SPAN;                   // lanes per group: 1, 2 or 4
    constexpr int NV = BF16 ? SPAN / 8 : SPAN / 4;  // 16-byte pieces of a span
    constexpr int PER_WORD = 32 / BITS;             // codes per 32-bit word
    constexpr int NWORDS = SPAN / PER_WORD;
    // what the constant upper bits of the rounded floats add up to in a packed word
    constexpr unsigned K = [] { unsigned k = 0; for (int i = 0; i < PER_WORD; ++i) k += kMagicBits << (BITS * i); return k; }();

    const unsigned chunk = blockIdx.x, h = blockIdx.y, b = blockIdx.z;          // grid (chunks of a row, heads, batch): no division
    const unsigned u0 = chunk * VAL_THREADS + threadIdx.x;                       // span within the row
    const unsigned n_row = (unsigned)p.T * (unsigned)p.ns;
    if (u0 - (threadIdx.x & 31) >= n_row) return;                                // the whole warp is past the row
    // whole groups are valid or not (spans per token are a multiple of LPG): the spare lanes of the row's last warp redo
    // its last span, take part in the shuffles and store nothing
    const bool valid = u0 < n_row;
    const unsigned u = valid ? u0 : n_row - 1;
    const unsigned tok = p.ns_shift >= 0 ? u >> p.ns_shift : u / (unsigned)p.ns;
    const unsigned sp = u - tok * (unsigned)p.ns;                                // span within the token
    const unsigned q = sp / LPG;                                                 // its group
    const long long in_off = (long long)b * p.sb + (long long)h * p.sh + (long long)tok * p.st + (long long)sp * SPAN;
    const long long out_tok = (long long)b * p.osb + (long long)h * p.osh + tok;

    uint4 raw[NV];
    {
        const uint4 *src = BF16 ? reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(p.v) + in_off)
                                : reinterpret_cast<const uint4 *>(reinterpret_cast<const float *>(p.v) + in_off);
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            raw[i] = make_uint4(0, 0, 0, 0);
            if (SQ_CHK_G(p.status, src + i, 16, p.x_v)) raw[i] = ldg128(src + i);
        }
    }
    // channel pair c (channels 2c, 2c + 1) as two floats, exact widening
    auto pair_of = [&](int c, float &x0, float &x1) {
        if (BF16) {
            const uint4 &r = raw[c >> 2];
            const unsigned w = (c & 3) == 0 ? r.x : (c & 3) == 1 ? r.y : (c & 3) == 2 ? r.z : r.w;
            x0 = bf16lo_to_f32(w);
            x1 = bf16hi_to_f32(w);
        } else {
            const uint4 &r = raw[c >> 1];
            x0 = __uint_as_float((c & 1) ? r.z : r.x);
            x1 = __uint_as_float((c & 1) ? r.w : r.y);
        }
    };

    // ---- min / max of the group
    float m, Mx;
    if (BF16) {
        unsigned mn2 = raw[0].x, mx2 = raw[0].x;                // packed bf16 pairs (exact), then across the pair
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const unsigned w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
#pragma unroll
            for (int k = (i == 0 ? 1 : 0); k < 4; ++k) { mn2 = hmin2_nan_bits(mn2, w[k]); mx2 = hmax2_nan_bits(mx2, w[k]); }
        }
        m = min_nan(bf16lo_to_f32(mn2), bf16hi_to_f32(mn2));
        Mx = max_nan(bf16lo_to_f32(mx2), bf16hi_to_f32(mx2));
    } else {
        float x0, x1;
        pair_of(0, x0, x1);
        m = min_nan(x0, x1);
        Mx = max_nan(x0, x1);
#pragma unroll
        for (int c = 1; c < SPAN / 2; ++c) {
            pair_of(c, x0, x1);
            m = min_nan(m, min_nan(x0, x1));
            Mx = max_nan(Mx, max_nan(x0, x1));
        }
    }

#pragma unroll
    for (int o = 1; o < LPG; o <<= 1) {                 // the group's other lanes
        m = min_nan(m, __shfl_xor_sync(0xffffffffu, m, o));
        Mx = max_nan(Mx, __shfl_xor_sync(0xffffffffu, Mx, o));
    }

    // ---- the grid
    const float rng = __fsub_rn(Mx, m);
    float delta = div_by_levels<BITS>(rng);
    if (!(rng > 0x1p-100f && rng < 0x1p100f)) delta = __fdiv_rn(rng, L);     // outside the range where that is exact: the division
    if (M16) {                                         // the stored binary16 values decide
        delta = __half2float(__float2half_rn(delta));
        m = __half2float(__float2half_rn(m));
    }
    const bool ok = delta > 0.0f && delta < __int_as_float(0x7f800000);
    const bool fast = delta > 0x1p-100f && delta < 0x1p100f;       // the hardware reciprocal is good to 1 ulp here
    float rcp;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(rcp) : "f"(delta));
    const float ra = __fmul_rn(rcp, 1.0f + 0x1p-20f), rb = __fmul_rn(rcp, 1.0f - 0x1p-20f);
    const u64 m2 = pk2(m, m), ra2 = pk2(ra, ra), rb2 = pk2(rb, rb), magic2 = pk2(kMagic, kMagic);

    // ---- codes: two channels per instruction (packed f32x2).  Both ends of the bracket are rounded and packed (added
    // up shifted into place); the ends differ by at most one level, upwards, so the difference of the two packed words
    // has exactly one bit set for every element that the fast path could not decide.
    constexpr unsigned ALL = [] { unsigned a = 0; for (int i = 0; i < PER_WORD; ++i) a |= 1u << (BITS * i); return a; }();
    uint32_t words[NWORDS];
#pragma unroll
    for (int wd = 0; wd < NWORDS; ++wd) {
        unsigned acc_a = 0u - K, acc_b = 0u - K;
#pragma unroll
        for (int k = 0; k < PER_WORD; k += 2) {
            float x0, x1, ya0, ya1, yb0, yb1;
            pair_of((wd * PER_WORD + k) / 2, x0, x1);
            const u64 dlt2 = sub2(pk2(x0, x1), m2);
            unpk2(fma2(dlt2, ra2, magic2), ya0, ya1);
            unpk2(fma2(dlt2, rb2, magic2), yb0, yb1);
            if (M16) {                                  // rounded metadata: t may leave [0, L]
                ya0 = fminf(fmaxf(ya0, kMagic), kMagic + L); yb0 = fminf(fmaxf(yb0, kMagic), kMagic + L);
                ya1 = fminf(fmaxf(ya1, kMagic), kMagic + L); yb1 = fminf(fmaxf(yb1, kMagic), kMagic + L);
            }
            acc_a += __float_as_uint(ya0) << (BITS * k);
            acc_a += __float_as_uint(ya1) << (BITS * (k + 1));
            acc_b += __float_as_uint(yb0) << (BITS * k);
            acc_b += __float_as_uint(yb1) << (BITS * (k + 1));
        }
        const unsigned undecided = fast ? acc_a - acc_b : ALL;
        if (undecided && ok) {
            const long long e0 = in_off + wd * PER_WORD;        // first element of this word
            const void *elems = BF16 ? static_cast<const void *>(reinterpret_cast<const __nv_bfloat16 *>(p.v) + e0)
                                     : static_cast<const void *>(reinterpret_cast<const float *>(p.v) + e0);
            acc_a = patch_word<BITS, BF16, M16>(acc_a, undecided, elems, m, delta, ra, rb, fast);
        }
        words[wd] = ok ? acc_a : 0u;                    // no grid (constant or non-finite group): codes 0
    }

    if (!valid) return;
    unsigned char *cp = p.codes + out_tok * p.row_bytes + (long long)sp * (SPAN * BITS / 8);
    const long long meta_idx = out_tok * p.ng + q;
    if (!SQ_CHK_G(p.status, cp, SPAN * BITS / 8, p.x_codes) ||
        !SQ_CHK_G(p.status, static_cast<char *>(p.scales) + meta_idx * (M16 ? 2 : 4), M16 ? 2 : 4, p.x_scales) ||
        !SQ_CHK_G(p.status, static_cast<char *>(p.zeros) + meta_idx * (M16 ? 2 : 4), M16 ? 2 : 4, p.x_zeros))
        return;
    if (NWORDS % 4 == 0) {
#pragma unroll
        for (int i = 0; i < NWORDS / 4; ++i)
            reinterpret_cast<uint4 *>(cp)[i] = make_uint4(words[4 * i], words[4 * i + 1], words[4 * i + 2], words[4 * i + 3]);
    } else {
#pragma unroll
        for (int i = 0; i < NWORDS / 2; ++i)
            reinterpret_cast<uint2 *>(cp)[i] = make_uint2(words[2 * i], words[2 * i + 1]);
    }
    if (LPG > 1 && (sp & (LPG - 1)) != 0) return;       // one lane per group stores its grid
    if (M16) {
        reinterpret_cast<__half *>(p.scales)[meta_idx] = __float2half_rn(delta);      // exact: already binary16 values
        reinterpret_cast<__half *>(p.zeros)[meta_idx] = __float2half_rn(m);
    } else {
        reinterpret_cast<float *>(p.scales)[meta_idx] = delta;
        reinterpret_cast<float *>(p.zeros)[meta_idx] = m;
    }
    if (!ok) atomicOr(p.status, delta == 0.0f ? SQUAT_FLAG_ZERO_RANGE : SQUAT_FLAG_NONFINITE);
}

// (x & MASK) | c as ONE three-input logic instruction (left to itself the compiler emits two)
template <uint32_t MASK>
__device__ __forceinline__ uint32_t and_or(uint32_t x, uint32_t c)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(x), "n"(MASK), "r"(c));
    return d;
}

// Channels (2 I, 2 I + 1) of a thread's 8 codes as two exact floats: each code, masked in place at bit position s, is OR-ed
// under the exponent of 2^(23 - s) (the pair `bias`, held in registers), which makes the word 2^(23 - s) + c; subtracting
// the bias leaves c.  4-bit codes of channels 4..7 sit in the upper half of the word (`hi` = word >> 16).
template <int BITS, int I>
__device__ __forceinline__ u64 codes_pair(uint32_t lo, uint32_t hi, u64 bias)
{
    constexpr int S0 = (BITS * 2 * I) % 16, S1 = (BITS * (2 * I + 1)) % 16;
    constexpr uint32_t FIELD = (1u << BITS) - 1u;
    const uint32_t word = (BITS == 4 && I >= 2) ? hi : lo;
    float b0, b1;
    unpk2(bias, b0, b1);
    const float f0 = __uint_as_float(and_or<(FIELD << S0)>(word, __float_as_uint(b0)));
    const float f1 = __uint_as_float(and_or<(FIELD << S1)>(word, __float_as_uint(b1)));
    return sub2(pk2(f0, f1), bias);
}

// Dequantizer.  One thread owns 8 consecutive channels (16 bytes of bf16 output, 32 of float32) of TOK = 4 or 8
// consecutive tokens of one key group, so the 8 scales and zeros of a key cache are read once for all of them (8 tokens
// on large inputs, 4 where that would leave SMs without work); the lanes of a warp cover whole tokens, so every store
// instruction writes full 256-byte rows.  A code becomes a float without shifting: its bits, masked in place at bit
// position s, are OR-ed under the exponent of 2^(23 - s), which makes the word 2^(23 - s) + c exactly; subtracting that
// power of two leaves c (both steps exact), then one fma: deq(c) = fma(c, scale, zero), rounded once.  Two channels per
// instruction (packed f32x2).
template <int BITS, bool KEYS, bool OUT_BF16, bool M16, int TOK>
__global__ void __launch_bounds__(256) dequant_kernel(
    const unsigned char *__restrict__ codes, const void *__restrict__ scales, const void *__restrict__ zeros,
    int per_tok_shift, int T, int d, int g_shift, long long isb, long long ish, long long isb_g, long long ish_g, void *__restrict__ out)
{
    // grid (chunks of a row, heads, batch).  per_tok_shift: log2 of the threads per token (d / 8, a power of two);
    // g_shift: log2 of the group size; isb_g, ish_g: the token strides divided by the group size (keys: group strides)
    constexpr int CH = 8;                                 // channels per thread
    const int slots = 256 >> per_tok_shift;               // token runs (TOK tokens each) per CTA
    const int row_bytes = d * BITS / 8;
    // bias pairs 2^(23 - s) for the bit positions s of channels (2 i, 2 i + 1); positions are taken modulo 16 for 4-bit
    // codes (the upper half of the word is shifted down first)
    u64 bias2[CH / 2];
#pragma unroll
    for (int i = 0; i < CH / 2; ++i) {
        const int s0 = (BITS * 2 * i) % 16, s1 = (BITS * (2 * i + 1)) % 16;
        bias2[i] = pk2(__uint_as_float((unsigned)(150 - s0) << 23), __uint_as_float((unsigned)(150 - s1) << 23));
        asm volatile("" : "+l"(bias2[i]));              // held in registers: the logic instruction below takes them from there
    }
    // one CTA = one chunk of slots * TOK tokens of one (batch, head) row; no division anywhere
    const unsigned chunk = blockIdx.x;
    const int h = (int)blockIdx.y;
    const long long b = blockIdx.z;
    const unsigned bh = blockIdx.z * gridDim.y + blockIdx.y;
    const int slot = (int)threadIdx.x >> per_tok_shift, c8 = (int)threadIdx.x - (slot << per_tok_shift);
    const int t0 = ((int)chunk * slots + slot) * TOK;
    if (slot < slots && t0 < T) {
        const long long in_tok0 = b * isb + h * ish;
        u64 sc2[CH / 2], zr2[CH / 2];
        if (KEYS) {
            const long long base = (b * isb_g + h * ish_g + (t0 >> g_shift)) * d + c8 * CH;
            if (M16) {
                const uint4 s8 = __ldg(reinterpret_cast<const uint4 *>(reinterpret_cast<const __half *>(scales) + base));
                const uint4 z8 = __ldg(reinterpret_cast<const uint4 *>(reinterpret_cast<const __half *>(zeros) + base));
                const uint32_t sw[4] = {s8.x, s8.y, s8.z, s8.w}, zw[4] = {z8.x, z8.y, z8.z, z8.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float2 sf = __half22float2(*reinterpret_cast<const __half2 *>(&sw[k]));
                    const float2 zf = __half22float2(*reinterpret_cast<const __half2 *>(&zw[k]));
                    sc2[k] = pk2(sf.x, sf.y);
                    zr2[k] = pk2(zf.x, zf.y);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const float4 s4 = __ldg(reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(scales) + base) + i);
                    const float4 z4 = __ldg(reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(zeros) + base) + i);
                    sc2[2 * i] = pk2(s4.x, s4.y); sc2[2 * i + 1] = pk2(s4.z, s4.w);
                    zr2[2 * i] = pk2(z4.x, z4.y); zr2[2 * i + 1] = pk2(z4.z, z4.w);
                }
            }
        }
        // the codes of the thread's tokens first (independent loads in flight), then the arithmetic
        // pointers of the first token; a step to the next token is one 32-bit stride (no 64-bit index arithmetic per token)
        const int nt = T - t0 < TOK ? T - t0 : TOK;             // tokens of this run that exist (fewer only at a row's end)
        const unsigned char *cp0 = codes + (in_tok0 + t0) * row_bytes + c8 * (CH * BITS / 8);
        const int mstep = d >> g_shift;                         // groups per token
        const long long mi0 = (in_tok0 + t0) * mstep + ((c8 * CH) >> g_shift);
        char *op0 = static_cast<char *>(out) + ((((long long)bh * T) + t0) * d + c8 * CH) * (OUT_BF16 ? 2 : 4);
        const int ostep = d * (OUT_BF16 ? 2 : 4);
        uint32_t cw[TOK];
#pragma unroll
        for (int tt = 0; tt < TOK; ++tt) {
            const unsigned char *cp = cp0 + (tt < nt ? tt : nt - 1) * row_bytes;
            cw[tt] = BITS == 2 ? (uint32_t)__ldg(reinterpret_cast<const uint16_t *>(cp)) : __ldg(reinterpret_cast<const uint32_t *>(cp));
        }
#pragma unroll
        for (int tt = 0; tt < TOK; ++tt) {
            if (tt >= nt) break;
            u64 s2 = 0, z2 = 0;
            if (!KEYS) {
                const long long mi = mi0 + tt * mstep;
                float s1, z1;
                if (M16) {
                    s1 = __half2float(__ldg(reinterpret_cast<const __half *>(scales) + mi));
                    z1 = __half2float(__ldg(reinterpret_cast<const __half *>(zeros) + mi));
                } else {
                    s1 = __ldg(reinterpret_cast<const float *>(scales) + mi);
                    z1 = __ldg(reinterpret_cast<const float *>(zeros) + mi);
                }
                s2 = pk2(s1, s1);
                z2 = pk2(z1, z1);
            }
            const uint32_t lo = cw[tt], hi = cw[tt] >> 16;        // 4-bit codes: channels 4..7 sit in the upper half
            u64 c2[CH / 2], y2[CH / 2];
            c2[0] = codes_pair<BITS, 0>(lo, hi, bias2[0]);
            c2[1] = codes_pair<BITS, 1>(lo, hi, bias2[1]);
            c2[2] = codes_pair<BITS, 2>(lo, hi, bias2[2]);
            c2[3] = codes_pair<BITS, 3>(lo, hi, bias2[3]);
#pragma unroll
            for (int i = 0; i < CH / 2; ++i) y2[i] = KEYS ? fma2(c2[i], sc2[i], zr2[i]) : fma2(c2[i], s2, z2);
            char *op_t = op0 + tt * ostep;
            if (OUT_BF16) {
                uint32_t pk[CH / 2];
#pragma unroll
                for (int i = 0; i < CH / 2; ++i) {
                    float a, b_;
                    unpk2(y2[i], a, b_);
                    __nv_bfloat162 p2 = __floats2bfloat162_rn(a, b_);
                    pk[i] = *reinterpret_cast<uint32_t *>(&p2);
                }
                *reinterpret_cast<uint4 *>(op_t) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            } else {
                float4 *op = reinterpret_cast<float4 *>(op_t);
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    float a, b_, c, e;
                    unpk2(y2[2 * i], a, b_);
                    unpk2(y2[2 * i + 1], c, e);
                    op[i] = make_float4(a, b_, c, e);
                }
            }
        }
    }
}

template <int G, int BITS, bool BF16, bool M16>
int launch_values_inst(const ValParams &p, long long rows, cudaStream_t st)
{
    quant_values_kernel<G, BITS, BF16, M16><<<dim3(p.chunks_per_row, (unsigned)p.H, (unsigned)(rows / p.H)), VAL_THREADS, 0, st>>>(p);
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return SQUAT_OK;
}

template <int G, int BITS>
int launch_values(const ValParams &p, long long rows, int dtype, int meta16, cudaStream_t st)
{
    if (dtype == SQUAT_BF16) return meta16 ? launch_values_inst<G, BITS, true, true>(p, rows, st) : launch_values_inst<G, BITS, true, false>(p, rows, st);
    return meta16 ? launch_values_inst<G, BITS, false, true>(p, rows, st) : launch_values_inst<G, BITS, false, false>(p, rows, st);
}

}  // namespace

int squat_launch_quant_values(const void *v, int dtype, int batch, int H, int T, int d,
                              long long sb, long long sh, long long st_, int bits, int G,
                              unsigned char *codes, void *scales, void *zeros,
                              long long osb, long long osh, unsigned *status, int meta16, cudaStream_t st)
{
    const long long rows = (long long)batch * H;
    if (rows == 0 || T == 0) return SQUAT_OK;
    ValParams p;
    if (d % 32 != 0) return SQUAT_ERR_SHAPE;
    p.v = v; p.H = H; p.T = T; p.ng = d / G; p.ns = d / 32;
    p.ns_shift = -1;
    for (int sft = 0; sft < 20; ++sft)
        if ((1 << sft) == p.ns) p.ns_shift = sft;
    const long long row_units = (long long)T * p.ns;
    const long long chunks = (row_units + VAL_THREADS - 1) / VAL_THREADS;
    if (row_units > 0x7fffffffLL || chunks > 0x7fffffffLL || H > 65535 || batch > 65535) return SQUAT_ERR_UNSUPPORTED;    // 32-bit span indices, grid limits
    p.chunks_per_row = (unsigned)chunks;
    p.sb = sb; p.sh = sh; p.st = st_;
    p.codes = codes; p.scales = scales; p.zeros = zeros; p.osb = osb; p.osh = osh;
    p.row_bytes = d * bits / 8;
    p.status = status;
#ifdef SQUAT_CHECKED
    {
        const unsigned long long es = dtype == SQUAT_BF16 ? 2 : 4, ms = meta16 ? 2 : 4;
        p.x_v = {v, (unsigned long long)((batch - 1) * sb + (H - 1) * sh + (long long)(T - 1) * st_ + d) * es};
        const unsigned long long toks = (unsigned long long)((batch - 1) * osb + (H - 1) * osh + T);
        p.x_codes = {codes, toks * p.row_bytes};
        p.x_scales = {scales, toks * p.ng * ms};
        p.x_zeros = {zeros, toks * p.ng * ms};
    }
#endif
#define SQ_V(GG, BB) return launch_values<GG, BB>(p, rows, dtype, meta16, st)
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
    const long long rows = (long long)batch * H;
    if (rows == 0 || T == 0) return SQUAT_OK;
    const int per_tok = d / 8;
    if (per_tok < 1 || per_tok > 256 || d % 8 != 0) return SQUAT_ERR_UNSUPPORTED;
    int per_tok_shift = -1, g_shift = -1;
    for (int sft = 0; sft < 9; ++sft) {
        if ((1 << sft) == per_tok) per_tok_shift = sft;
        if ((1 << sft) == G) g_shift = sft;
    }
    if (per_tok_shift < 0 || g_shift < 0) return SQUAT_ERR_UNSUPPORTED;          // d / 8 and the group size are powers of two
    if (kind == SQUAT_KEYS && (isb % G != 0 || ish % G != 0)) return SQUAT_ERR_SHAPE;    // key groups do not straddle rows
    const int slots = 256 / per_tok;
    // 8 tokens per thread where that still gives every SM several CTAs, else 4
    const long long chunks8 = (T + slots * 8 - 1) / (slots * 8);
    const bool tok8 = rows * chunks8 >= (long long)sms * 16;
    const long long chunks = tok8 ? chunks8 : (T + slots * 4 - 1) / (slots * 4);
    if (chunks > 0x7fffffffLL || H > 65535 || batch > 65535) return SQUAT_ERR_UNSUPPORTED;
    const dim3 grid((unsigned)chunks, (unsigned)H, (unsigned)batch);
#define SQ_D1(BB, KK, OO, MM, TT) dequant_kernel<BB, KK, OO, MM, TT><<<grid, 256, 0, st>>>(codes, scales, zeros, per_tok_shift, T, d, g_shift, isb, ish, isb / G, ish / G, out)
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
