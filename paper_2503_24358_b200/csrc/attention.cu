// Reader of the packed cache: one decode step of attention (Section 2, "(Masked) Attention mechanism";
// the score vector w^deq = <q, deq(k_i)> / sqrt(d) of the proof of Theorem 1; the most recent tokens come
// from the full-precision residual buffer of Algorithm 1).
//
//   out_hq = softmax_i( s <q_hq, k_i> ) . v_i ,   k_i, v_i = dequantized cache rows, then the residual rows
//
// The cache is never dequantized to memory.  Per-channel key metadata folds into the query: for the G tokens
// that share (scale_c, zero_c),  <q, deq(k_t)> = sum_c (q_c scale_c) code_tc + sum_c q_c zero_c, so a group
// costs one scaled copy of the query and each token one dot product with its 128 codes.  Per-token value
// metadata folds into the weight: p_t deq(v_t)_c = (p_t scale_tg) code_tc + p_t zero_tg.  Codes become floats
// without a conversion: the code bits are shifted under the top of a float's mantissa, giving 1 + code / 2^bits
// exactly (two integer instructions); the "1 +" is taken out again through one constant per group.
//
// attn_partial_kernel   grid (token chunks of 256..1024 x query-head passes, KV heads, batch).  Key phase: a warp takes
//                       32 tokens (lane = token, its codes are 2 or 4 128-bit loads), scores go to shared
//                       memory.  Then the chunk's maximum and exp().  Value phase: a warp reads 128 bytes of
//                       codes per step (lane = one 32-bit word of one of 4 or 2 tokens) and accumulates
//                       weight x code for its channels.  Writes (unnormalised sum, max, denominator) per chunk.
// attn_combine_kernel   grid (query heads, batch): adds the residual buffer's tokens (plain fp32 dot products)
//                       and merges the chunks with the usual max / denominator rescaling.
//
// Bound: HBM (bits/8 + metadata bytes per cached element); the unpacking arithmetic is close behind.
//
// Keys stored BEFORE the rotary position embedding (Section 4, the "pre" variant): the reader applies the
// embedding on the fly.  Token t of the cache sits at position P = first_pos + t; channel pair (i, i + 64) of its
// dequantized key turns by the angle P * base^(-2i/128).  With P = 32 a + l the turn is the product of a block
// turn (32 a theta_i: the same for the 32 tokens of a warp step, so it is applied to the query instead, with the
// opposite sign) and a lane turn (l theta_i: a table in shared memory, one entry per lane and pair).  Cosines and
// sines come from two tables the host fills in float64 (squat_rope_table_fill); the kernel only multiplies.  The
// key metadata cannot be folded into the query on this path: each pair is dequantized (one FMA per element),
// turned (4) and multiplied with the block-turned query of every head (2 per head).
#include "squat_internal.cuh"
#include <type_traits>
#include <cuda_fp16.h>

namespace {

constexpr int D = SQUAT_D;
constexpr int AT_THREADS = 256;
constexpr int AT_WARPS = AT_THREADS / 32;
constexpr int AT_CHUNK = 1024;            // most tokens per CTA (the launcher takes 256, 512 or 1024: enough CTAs to fill the GPU)

struct AttnParams {
    const void *q;             // [B, Hq, D]
    int q_bf16;
    int B, Hq, H, T;           // T: quantized tokens per (batch, head)
    const unsigned char *kc, *vc;
    const void *ks, *kz, *vs, *vz;   // float32, or binary16 in the M16 instances
    long long csb, csh;        // cache strides in tokens
    int G;
    const void *k_res, *v_res; // [B, H, R, D]
    int res_bf16, R;
    float scale;
    float *part;               // [B, Hq, nchunk, D]
    float *ml;                 // [B, Hq, nchunk, 2]
    int nchunk, chunk;         // chunk: tokens per CTA, a multiple of 256
    float *out;                // [B, Hq, D]
    // rotary tables (pre-embedding key storage only): cos/sin of (32 a theta_i) [blocks][64] and of (l theta_i) [32][64]
    const float2 *rope_a, *rope_b;
    long long first_pos;       // position of cached token 0; a multiple of 32
    int meta16;                // the cache's scales and zero-points are binary16
};

// 1 + code / 2^BITS as a float, for the code at position i of a 32-bit word (low bits first)
// A constant the compiler has to keep in a register: `(x & mask) | constant` is then ONE three-input logic instruction
// (mask as its immediate); with both as immediates it takes two, and the unpacking below is what fills the integer pipe.
// (x & MASK) | c as one three-input logic instruction
template <uint32_t MASK>
__device__ __forceinline__ uint32_t and_or(uint32_t x, uint32_t c)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(x), "n"(MASK), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t in_register(uint32_t v)
{
    uint32_t r;
    asm volatile("mov.b32 %0, %1;" : "=r"(r) : "r"(v));
    return r;
}
// one_bits: the bit pattern of 1.0f, held in a register (in_register)
template <int BITS>
__device__ __forceinline__ float code_as_float(uint32_t w, int i, uint32_t one_bits)
{
    constexpr int TOP = 23 - BITS;                              // the code's low bit lands here
    constexpr uint32_t MASK = ((1u << BITS) - 1u) << TOP;
    const int pos = BITS * i;
    uint32_t sh = pos <= TOP ? (w << (TOP - pos)) : (w >> (pos - TOP));
    asm("" : "+r"(sh));                                        // keep the shift where it is (not re-associated behind the mask)
    return __uint_as_float(and_or<MASK>(sh, one_bits));
}

// Two neighbouring 2-bit codes (positions 2 j and 2 j + 1 of a word) as floats with ONE shift: their 4-bit window goes
// to mantissa bits 19..22.  The upper code, under the exponent of 1, reads 1 + c/4; the lower one, two mantissa bits
// further down, is put under the exponent of 4 and reads 4 + c/4 -- the same step per level, a different constant,
// which goes into the per-group constant like the "1 +".
// one_bits, four_bits: the bit patterns of 1.0f and 4.0f, held in registers (in_register)
__device__ __forceinline__ void code_pair_as_floats(uint32_t w, int j, float &f_even, float &f_odd, uint32_t one_bits, uint32_t four_bits)
{
    const int pos = 4 * j;
    uint32_t sh = pos <= 19 ? (w << (19 - pos)) : (w >> (pos - 19));
    asm("" : "+r"(sh));                                        // one shift for both codes: not re-associated behind the masks
    f_even = __uint_as_float(and_or<0x00180000u>(sh, four_bits));
    f_odd = __uint_as_float(and_or<0x00600000u>(sh, one_bits));
}
typedef unsigned long long u64;
__device__ __forceinline__ u64 pack2f(float lo, float hi)
{
    u64 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ u64 ffma2(u64 a, u64 b, u64 c)
{
    u64 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ float sum2f(u64 v)
{
    float lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
    return lo + hi;
}

__device__ __forceinline__ float warp_sum_f(float v)
{
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
    return v;
}
__device__ __forceinline__ float warp_max_f(float v)
{
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, m));
    return v;
}

__device__ __forceinline__ float load_elem(const void *p, long long idx, int bf16)
{
    if (bf16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(p)[idx]);
    return reinterpret_cast<const float *>(p)[idx];
}

// scale / zero-point element i of a metadata array stored as float32 or binary16
template <bool M16>
__device__ __forceinline__ float meta_at(const void *p, long long i)
{
    if (M16) return __half2float(__ldg(reinterpret_cast<const __half *>(p) + i));
    return __ldg(reinterpret_cast<const float *>(p) + i);
}
// four consecutive elements starting at i (a multiple of 4)
template <bool M16>
__device__ __forceinline__ float4 meta4_at(const void *p, long long i)
{
    if (M16) {
        const uint2 r = __ldg(reinterpret_cast<const uint2 *>(reinterpret_cast<const __half *>(p) + i));
        const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&r.x));
        const float2 b = __half22float2(*reinterpret_cast<const __half2 *>(&r.y));
        return make_float4(a.x, a.y, b.x, b.y);
    }
    return __ldg(reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(p) + i));
}

template <int BITS, int NQ, bool ROPE, bool M16>
__global__ void __launch_bounds__(AT_THREADS, NQ >= 4 ? (ROPE ? 2 : 3) : (ROPE ? 3 : 4)) attn_partial_kernel(const AttnParams p)
{
    constexpr int WPT = D * BITS / 32;                          // 32-bit words per token: 8 or 16
    constexpr int CPW = 32 / BITS;                              // codes per word: 16 or 8
    constexpr float LV = float(1 << BITS);
    constexpr bool PAIRS = BITS == 2 && NQ <= 2;                // two codes per shift and packed multiply-adds (code_pair_as_floats)
    const uint32_t one_bits = in_register(0x3F800000u), four_bits = in_register(0x40800000u);
    extern __shared__ __align__(16) float sm[];
    float *qsm = sm;                                            // [NQ][D]      q * softmax scale
    float *qs = qsm + NQ * D;                                   // [warps][NQ][D] query x key scale x 2^BITS of the warp's group
    float *sc = qs + AT_WARPS * NQ * D;                         // [NQ][AT_CHUNK] scores, then weights
    float *red = sc + NQ * AT_CHUNK;                            // [NQ][warps] and [NQ] scratch of the reductions
    float2 *lane_turn = reinterpret_cast<float2 *>(red + NQ * AT_WARPS + 8);   // ROPE: [64][32] cos/sin of (lane theta_i)
    float4 *sz_all = reinterpret_cast<float4 *>(lane_turn + 64 * 32);           // ROPE: [warps][64] (S_i, Z_i, S_{i+64}, Z_{i+64})
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chunk = blockIdx.x % p.nchunk, qpass = blockIdx.x / p.nchunk;
    const int h = blockIdx.y, b = blockIdx.z;
    const int qpk = p.Hq / p.H;
    const int hq0 = h * qpk + qpass * NQ;
    const int nq_here = min(NQ, qpk - qpass * NQ);
    const int t0 = chunk * p.chunk, t1 = min(p.T, t0 + p.chunk);
    const long long ctok0 = (long long)b * p.csb + (long long)h * p.csh;

    for (int i = tid; i < NQ * D; i += AT_THREADS) {
        const int qi = i / D, c = i % D;
        qsm[i] = qi < nq_here ? p.scale * load_elem(p.q, ((long long)b * p.Hq + hq0 + qi) * D + c, p.q_bf16) : 0.0f;
    }
    if (ROPE) {
        for (int i = tid; i < 64 * 32; i += AT_THREADS) lane_turn[i] = __ldg(p.rope_b + (i & 31) * 64 + (i >> 5));   // [pair][lane]
    }
    __syncthreads();

    // ---------------------------------------------------------------- key phase: scores
    float *qsw = qs + warp * NQ * D;
    for (int blk = t0 + 32 * warp; blk < t1; blk += 32 * AT_WARPS) {
        const long long mrow = (ctok0 / p.G + blk / p.G) * D;
        if (ROPE) {
            // ---- keys stored before the rotary embedding
            const long long a_blk = (p.first_pos + blk) >> 5;          // block turn: the same for the warp's 32 tokens
            float2 *qb = reinterpret_cast<float2 *>(qsw);              // [NQ][64]: the heads' queries turned back by the block turn
            float4 *sz = sz_all + warp * 64;
            // this lane's token's codes first: their latency overlaps the tables' and the metadata's
            const uint4 *cp = reinterpret_cast<const uint4 *>(p.kc + (ctok0 + blk + lane) * (long long)(D * BITS / 8));
            uint32_t wd[WPT];
#pragma unroll
            for (int v4 = 0; v4 < WPT / 4; ++v4) {
                const uint4 cw = __ldg(cp + v4);
                wd[4 * v4] = cw.x; wd[4 * v4 + 1] = cw.y; wd[4 * v4 + 2] = cw.z; wd[4 * v4 + 3] = cw.w;
            }
            __syncwarp();
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int i = lane + 32 * hh;
                const float2 cs = __ldg(p.rope_a + a_blk * 64 + i);
#pragma unroll
                for (int qi = 0; qi < NQ; ++qi) {
                    const float q0 = qsm[qi * D + i], q1 = qsm[qi * D + i + 64];
                    qb[qi * 64 + i] = make_float2(fmaf(q0, cs.x, q1 * cs.y), fmaf(q1, cs.x, -q0 * cs.y));
                }
                const float s0 = meta_at<M16>(p.ks, mrow + i) * LV, s1 = meta_at<M16>(p.ks, mrow + i + 64) * LV;
                sz[i] = make_float4(s0, meta_at<M16>(p.kz, mrow + i) - s0, s1, meta_at<M16>(p.kz, mrow + i + 64) - s1);
            }
            __syncwarp();
            float acc[NQ][2];
#pragma unroll
            for (int qi = 0; qi < NQ; ++qi) acc[qi][0] = acc[qi][1] = 0.0f;
#pragma unroll
            for (int wi = 0; wi < WPT / 2; ++wi)
#pragma unroll
                for (int pos = 0; pos < CPW; ++pos) {
                    const int i = wi * CPW + pos;                       // pair (i, i + 64): same code position, WPT / 2 words apart
                    const float4 m4 = sz[i];
                    const float k0 = fmaf(code_as_float<BITS>(wd[wi], pos, one_bits), m4.x, m4.y);
                    const float k1 = fmaf(code_as_float<BITS>(wd[wi + WPT / 2], pos, one_bits), m4.z, m4.w);
                    const float2 cs = lane_turn[i * 32 + lane];
                    const float r0 = fmaf(k0, cs.x, -k1 * cs.y), r1 = fmaf(k0, cs.y, k1 * cs.x);
#pragma unroll
                    for (int qi = 0; qi < NQ; ++qi) {
                        const float2 qq = qb[qi * 64 + i];
                        acc[qi][pos & 1] = fmaf(r1, qq.y, fmaf(r0, qq.x, acc[qi][pos & 1]));
                    }
                }
#pragma unroll
            for (int qi = 0; qi < NQ; ++qi) sc[qi * AT_CHUNK + blk - t0 + lane] = acc[qi][0] + acc[qi][1];
            continue;
        }
        const float4 s4 = meta4_at<M16>(p.ks, mrow + 4 * lane);
        const float4 z4 = meta4_at<M16>(p.kz, mrow + 4 * lane);
        // this lane's token's codes: asked for before the metadata are worked on, so that the two loads' latencies overlap
        const uint4 *cp = reinterpret_cast<const uint4 *>(p.kc + (ctok0 + blk + lane) * (long long)(D * BITS / 8));
        uint4 cwv[WPT / 4];
#pragma unroll
        for (int v4 = 0; v4 < WPT / 4; ++v4) cwv[v4] = __ldg(cp + v4);
        float k0[NQ];
        __syncwarp();
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi) {
            const float4 qv = *reinterpret_cast<const float4 *>(qsm + qi * D + 4 * lane);
            const float4 v = make_float4(qv.x * s4.x * LV, qv.y * s4.y * LV, qv.z * s4.z * LV, qv.w * s4.w * LV);
            *reinterpret_cast<float4 *>(qsw + qi * D + 4 * lane) = v;
            const float zs = qv.x * z4.x + qv.y * z4.y + qv.z * z4.z + qv.w * z4.w;
            // sum_c q_c zero_c - sum_c qs'_c bias_c takes the codes' constants out again: "1 +", or for 2-bit codes
            // "4 +" on even and "1 +" on odd channels (code_pair_as_floats)
            k0[qi] = PAIRS ? warp_sum_f(zs - (4.0f * v.x + v.y + 4.0f * v.z + v.w)) : warp_sum_f(zs - (v.x + v.y + v.z + v.w));
        }
        __syncwarp();
        if (PAIRS) {
            // two channels per instruction: (f_even, f_odd) x (q'_even, q'_odd) into two packed accumulators per head
            u64 acc2[NQ][2];
#pragma unroll
            for (int qi = 0; qi < NQ; ++qi) acc2[qi][0] = acc2[qi][1] = 0ull;
#pragma unroll
            for (int v4 = 0; v4 < WPT / 4; ++v4) {
                const uint4 cw = cwv[v4];
                const uint32_t w4[4] = {cw.x, cw.y, cw.z, cw.w};
#pragma unroll
                for (int wi = 0; wi < 4; ++wi)
#pragma unroll
                    for (int i4 = 0; i4 < CPW / 4; ++i4) {
                        const int ch = (v4 * 4 + wi) * CPW + 4 * i4;
                        float f0, f1, f2, f3;
                        code_pair_as_floats(w4[wi], 2 * i4, f0, f1, one_bits, four_bits);
                        code_pair_as_floats(w4[wi], 2 * i4 + 1, f2, f3, one_bits, four_bits);
                        const u64 fa = pack2f(f0, f1), fb = pack2f(f2, f3);
#pragma unroll
                        for (int qi = 0; qi < NQ; ++qi) {
                            const ulonglong2 qq = *reinterpret_cast<const ulonglong2 *>(qsw + qi * D + ch);
                            acc2[qi][0] = ffma2(fa, qq.x, acc2[qi][0]);
                            acc2[qi][1] = ffma2(fb, qq.y, acc2[qi][1]);
                        }
                    }
            }
#pragma unroll
            for (int qi = 0; qi < NQ; ++qi)
                sc[qi * AT_CHUNK + blk - t0 + lane] = (sum2f(acc2[qi][0]) + sum2f(acc2[qi][1])) + k0[qi];
        } else {
        float acc[NQ][4];                                      // four partial sums per query head: independent FMA chains
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi) acc[qi][0] = acc[qi][1] = acc[qi][2] = acc[qi][3] = 0.0f;
#pragma unroll
        for (int v4 = 0; v4 < WPT / 4; ++v4) {
            const uint4 cw = cwv[v4];
            const uint32_t w4[4] = {cw.x, cw.y, cw.z, cw.w};
#pragma unroll
            for (int wi = 0; wi < 4; ++wi)
#pragma unroll
                for (int i4 = 0; i4 < CPW / 4; ++i4) {
                    const int ch = (v4 * 4 + wi) * CPW + 4 * i4;
                    const float f0 = code_as_float<BITS>(w4[wi], 4 * i4, one_bits), f1 = code_as_float<BITS>(w4[wi], 4 * i4 + 1, one_bits),
                                f2 = code_as_float<BITS>(w4[wi], 4 * i4 + 2, one_bits), f3 = code_as_float<BITS>(w4[wi], 4 * i4 + 3, one_bits);
#pragma unroll
                    for (int qi = 0; qi < NQ; ++qi) {
                        const float4 qq = *reinterpret_cast<const float4 *>(qsw + qi * D + ch);
                        acc[qi][0] = fmaf(f0, qq.x, acc[qi][0]);
                        acc[qi][1] = fmaf(f1, qq.y, acc[qi][1]);
                        acc[qi][2] = fmaf(f2, qq.z, acc[qi][2]);
                        acc[qi][3] = fmaf(f3, qq.w, acc[qi][3]);
                    }
                }
        }
#pragma unroll
        for (int qi = 0; qi < NQ; ++qi)
            sc[qi * AT_CHUNK + blk - t0 + lane] = ((acc[qi][0] + acc[qi][1]) + (acc[qi][2] + acc[qi][3])) + k0[qi];
        }
    }
    __syncthreads();

    // ---------------------------------------------------------------- chunk maximum, weights, denominator
    const int nt = t1 - t0;
    float mx[NQ], den[NQ];
#pragma unroll
    for (int qi = 0; qi < NQ; ++qi) {
        float m = -INFINITY;
        for (int i = tid; i < nt; i += AT_THREADS) m = fmaxf(m, sc[qi * AT_CHUNK + i]);
        m = warp_max_f(m);
        if (lane == 0) red[qi * AT_WARPS + warp] = m;
    }
    __syncthreads();
#pragma unroll
    for (int qi = 0; qi < NQ; ++qi) {
        float m = red[qi * AT_WARPS];
#pragma unroll
        for (int w = 1; w < AT_WARPS; ++w) m = fmaxf(m, red[qi * AT_WARPS + w]);
        mx[qi] = m;
    }
    __syncthreads();
#pragma unroll
    for (int qi = 0; qi < NQ; ++qi) {
        float s = 0.0f;
        for (int i = tid; i < nt; i += AT_THREADS) {
            const float e = expf(sc[qi * AT_CHUNK + i] - mx[qi]);
            sc[qi * AT_CHUNK + i] = e;
            s += e;
        }
        s = warp_sum_f(s);
        if (lane == 0) red[qi * AT_WARPS + warp] = s;
    }
    __syncthreads();
#pragma unroll
    for (int qi = 0; qi < NQ; ++qi) {
        float s = 0.0f;
#pragma unroll
        for (int w = 0; w < AT_WARPS; ++w) s += red[qi * AT_WARPS + w];
        den[qi] = s;
    }

    // ---------------------------------------------------------------- value phase: sum_t weight_t deq(v_t)
    constexpr int TPI = 32 / WPT;                               // tokens per warp step: 4 or 2
    const int ts = lane / WPT, j = lane % WPT;
    const int ng = D / p.G, gidx = (j * CPW) / p.G;
    // packed pairs (even channel, odd channel); corr takes the codes' constants out: "1 +", or for 2-bit codes "4 +" on even
    // and "1 +" on odd channels (code_pair_as_floats)
    u64 accv2[NQ][CPW / 2];                                    // PAIRS
    float accv[NQ][CPW];                                        // otherwise
    float corr[NQ], corr_even[NQ];
#pragma unroll
    for (int qi = 0; qi < NQ; ++qi) {
        corr[qi] = corr_even[qi] = 0.0f;
#pragma unroll
        for (int i = 0; i < CPW / 2; ++i) accv2[qi][i] = 0ull;
#pragma unroll
        for (int i = 0; i < CPW; ++i) accv[qi][i] = 0.0f;
    }
    const int vtok = p.chunk / AT_WARPS;
    const int vbase = t0 + warp * vtok;
    const int vend = min(t1, vbase + vtok);
    const uint32_t *vcw = reinterpret_cast<const uint32_t *>(p.vc);
    auto vstep = [&](int tk, uint32_t w, float vs_raw, float vzr) {
        const float vsc = vs_raw * LV;
        if (PAIRS) {
            u64 a2[NQ];
#pragma unroll
            for (int qi = 0; qi < NQ; ++qi) {
                const float pw = sc[qi * AT_CHUNK + tk - t0];
                const float a = pw * vsc, pz = pw * vzr;
                a2[qi] = pack2f(a, a);
                corr[qi] += pz - a;
                corr_even[qi] += fmaf(-4.0f, a, pz);
            }
#pragma unroll
            for (int i = 0; i < CPW / 2; ++i) {
                float fe, fo;
                code_pair_as_floats(w, i, fe, fo, one_bits, four_bits);
                const u64 f2 = pack2f(fe, fo);
#pragma unroll
                for (int qi = 0; qi < NQ; ++qi) accv2[qi][i] = ffma2(f2, a2[qi], accv2[qi][i]);
            }
        } else {
            float a[NQ];
#pragma unroll
            for (int qi = 0; qi < NQ; ++qi) {
                const float pw = sc[qi * AT_CHUNK + tk - t0];
                a[qi] = pw * vsc;
                corr[qi] += pw * vzr - a[qi];
            }
#pragma unroll
            for (int i = 0; i < CPW; ++i) {
                const float f = code_as_float<BITS>(w, i, one_bits);
#pragma unroll
                for (int qi = 0; qi < NQ; ++qi) accv[qi][i] = fmaf(f, a[qi], accv[qi][i]);
            }
        }
    };
    int tk = vbase + ts;
    for (; tk + TPI < vend; tk += 2 * TPI) {                    // two steps' loads in flight before either is used
        const long long c0 = ctok0 + tk, c1 = c0 + TPI;
        const uint32_t w0 = __ldg(vcw + c0 * WPT + j), w1 = __ldg(vcw + c1 * WPT + j);
        const float s0 = meta_at<M16>(p.vs, c0 * ng + gidx), z0 = meta_at<M16>(p.vz, c0 * ng + gidx);
        const float s1 = meta_at<M16>(p.vs, c1 * ng + gidx), z1 = meta_at<M16>(p.vz, c1 * ng + gidx);
        vstep(tk, w0, s0, z0);
        vstep(tk + TPI, w1, s1, z1);
    }
    if (tk < vend) {
        const long long c0 = ctok0 + tk;
        vstep(tk, __ldg(vcw + c0 * WPT + j), meta_at<M16>(p.vs, c0 * ng + gidx), meta_at<M16>(p.vz, c0 * ng + gidx));
    }
    // add the group constant, fold the token classes of the warp, then the warps
    __syncthreads();                                            // everybody is done reading sc: reuse it as [warps][NQ][D]
    float *part_sm = sc;
#pragma unroll
    for (int qi = 0; qi < NQ; ++qi)
#pragma unroll
        for (int i = 0; i < CPW; ++i) {
            float v;
            if (PAIRS) {
                float lo_, hi_;
                asm("mov.b64 {%0, %1}, %2;" : "=f"(lo_), "=f"(hi_) : "l"(accv2[qi][i / 2]));
                v = (i & 1) ? hi_ + corr[qi] : lo_ + corr_even[qi];
            } else {
                v = accv[qi][i] + corr[qi];
            }
#pragma unroll
            for (int m = WPT; m < 32; m <<= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
            if (ts == 0) part_sm[(warp * NQ + qi) * D + j * CPW + i] = v;
        }
    __syncthreads();
    for (int i = tid; i < NQ * D; i += AT_THREADS) {
        const int qi = i / D, c = i % D;
        if (qi >= nq_here) continue;
        float s = 0.0f;
#pragma unroll
        for (int w = 0; w < AT_WARPS; ++w) s += part_sm[(w * NQ + qi) * D + c];
        p.part[(((long long)b * p.Hq + hq0 + qi) * p.nchunk + chunk) * D + c] = s;
    }
    if (tid < nq_here) {
        float *ml = p.ml + (((long long)b * p.Hq + hq0 + tid) * p.nchunk + chunk) * 2;
        ml[0] = mx[tid];
        ml[1] = den[tid];
    }
}

// One CTA per (batch, query head): the residual buffer's tokens, then the merge of the chunks.  The kernel is a chain
// of dependent global loads (residual keys -> scores -> weights -> residual values, chunk partials), so it is laid out
// for loads in flight rather than for arithmetic: 16 warps; a warp takes every 16th residual key row (8 at most, all
// loaded before the first is used); the value rows and the chunks are dealt to four groups of 128 threads (thread =
// channel) whose partial sums meet in shared memory.
constexpr int CB_THREADS = 512;
constexpr int CB_WARPS = CB_THREADS / 32;
constexpr int CB_GROUPS = CB_THREADS / D;
template <bool RES_BF16>
__global__ void __launch_bounds__(CB_THREADS, RES_BF16 ? 2 : 1) attn_combine_kernel(const AttnParams p)
{
    using row_t = typename std::conditional<RES_BF16, uint2, float4>::type;      // four channels of a residual row as loaded
    auto as_f4 = [](const row_t &r) {
        if constexpr (RES_BF16) return make_float4(bf16lo_to_f32(r.x), bf16hi_to_f32(r.x), bf16lo_to_f32(r.y), bf16hi_to_f32(r.y));
        else return r;
    };
    __shared__ float qv[D];
    __shared__ float w[SQUAT_ATTN_MAX_RESIDUAL];
    __shared__ float red[CB_WARPS];
    __shared__ float acc_sm[CB_GROUPS][D];
    __shared__ float den_sm[CB_GROUPS];
    __shared__ __align__(16) float vacc_sm[CB_WARPS][D];                  // the warps' weighted sums of their residual value rows
    __shared__ float vden_sm[CB_WARPS];
    const int hq = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
    const int c = tid % D, grp = tid / D;
    const int warp = tid >> 5, lane = tid & 31;
    const int h = hq / (p.Hq / p.H);
    if (tid < D) qv[tid] = p.scale * load_elem(p.q, ((long long)b * p.Hq + hq) * D + tid, p.q_bf16);
    __syncthreads();
    const long long rbase = ((long long)b * p.H + h) * p.R * D;
    const float *ml = p.ml + ((long long)b * p.Hq + hq) * p.nchunk * 2;
    const float *part = p.part + ((long long)b * p.Hq + hq) * p.nchunk * D;
    // Every global load of the kernel is issued before the first result is needed: the residual key rows, the residual
    // value rows (same rows per warp, same four channels per lane) and the first CB_PART chunk partials of every thread.
    constexpr int CB_ROWS = SQUAT_ATTN_MAX_RESIDUAL / CB_WARPS;           // 8 residual rows per warp
    constexpr int CB_PART = 4;                                            // chunks per thread held in registers (16 per CTA pass)
    row_t kraw[CB_ROWS], vraw[CB_ROWS];
    float pr[CB_PART];
    float2 pml[CB_PART];
    // scores of the residual rows: a lane takes 4 neighbouring channels (one 8- or 16-byte load), so a row is read as one
    // contiguous piece
    {
        const float4 q4 = *reinterpret_cast<const float4 *>(qv + 4 * lane);
        constexpr int ROWS = SQUAT_ATTN_MAX_RESIDUAL / CB_WARPS;          // 8
#pragma unroll
        for (int i = 0; i < ROWS; ++i) {
            const int t = warp + CB_WARPS * i;
            kraw[i] = row_t{};
            vraw[i] = row_t{};
            if (t < p.R) {
                if constexpr (RES_BF16) {
                    kraw[i] = __ldg(reinterpret_cast<const uint2 *>(reinterpret_cast<const __nv_bfloat16 *>(p.k_res) + rbase + (long long)t * D) + lane);
                    vraw[i] = __ldg(reinterpret_cast<const uint2 *>(reinterpret_cast<const __nv_bfloat16 *>(p.v_res) + rbase + (long long)t * D) + lane);
                } else {
                    kraw[i] = __ldg(reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(p.k_res) + rbase + (long long)t * D) + lane);
                    vraw[i] = __ldg(reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(p.v_res) + rbase + (long long)t * D) + lane);
                }
            }
        }
        // the chunks' partial sums and (max, denominator) pairs do not wait for the scores either
#pragma unroll
        for (int i = 0; i < CB_PART; ++i) {
            const int sidx = grp + CB_GROUPS * i;
            pr[i] = sidx < p.nchunk ? part[(long long)sidx * D + c] : 0.0f;
            pml[i] = sidx < p.nchunk ? *reinterpret_cast<const float2 *>(ml + 2 * sidx) : make_float2(-INFINITY, 0.0f);
        }
#pragma unroll
        for (int i = 0; i < ROWS; ++i) {
            const int t = warp + CB_WARPS * i;
            if (t >= p.R) break;                                           // warp-uniform
            float4 k4 = as_f4(kraw[i]);
            if (p.rope_a) {
                // residual rows are stored before the rotary embedding too: turn row t at position first_pos + T + t.
                // Lane l < 16 holds channels 4 l .. 4 l + 3, lane l + 16 their partners 64 channels up.
                const long long pos = p.first_pos + p.T + t;
                const float4 o4 = make_float4(__shfl_xor_sync(0xffffffffu, k4.x, 16), __shfl_xor_sync(0xffffffffu, k4.y, 16),
                                              __shfl_xor_sync(0xffffffffu, k4.z, 16), __shfl_xor_sync(0xffffffffu, k4.w, 16));
                const float sign = lane < 16 ? -1.0f : 1.0f;
                const float own[4] = {k4.x, k4.y, k4.z, k4.w}, oth[4] = {o4.x, o4.y, o4.z, o4.w};
                float rot[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int i2 = 4 * (lane & 15) + e;
                    const float2 ca = __ldg(p.rope_a + (pos >> 5) * 64 + i2), cb = __ldg(p.rope_b + (pos & 31) * 64 + i2);
                    const float cc = fmaf(ca.x, cb.x, -ca.y * cb.y), ss = fmaf(ca.y, cb.x, ca.x * cb.y);
                    rot[e] = fmaf(own[e], cc, sign * oth[e] * ss);
                }
                k4 = make_float4(rot[0], rot[1], rot[2], rot[3]);
            }
            const float sdot = warp_sum_f(fmaf(q4.x, k4.x, fmaf(q4.y, k4.y, fmaf(q4.z, k4.z, q4.w * k4.w))));
            if (lane == 0) w[t] = sdot;
        }
    }
    __syncthreads();
    float m = tid < p.R ? w[tid] : -INFINITY;
#pragma unroll
    for (int i = 0; i < CB_PART; ++i) m = fmaxf(m, pml[i].x);
    for (int sidx = grp + CB_GROUPS * CB_PART; sidx < p.nchunk; sidx += CB_GROUPS) m = fmaxf(m, ml[2 * sidx]);
    m = warp_max_f(m);
    if (lane == 0) red[warp] = m;
    __syncthreads();
    m = red[0];
#pragma unroll
    for (int i = 1; i < CB_WARPS; ++i) m = fmaxf(m, red[i]);
    __syncthreads();
    if (tid < p.R) w[tid] = expf(w[tid] - m);
    __syncthreads();
    // residual rows: warp `warp` holds rows warp, warp + 16, ... (channels 4 lane .. 4 lane + 3); the warps' sums meet in shared memory
    {
        float4 a4 = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        float dw = 0.0f;
#pragma unroll
        for (int i = 0; i < CB_ROWS; ++i) {
            const int t = warp + CB_WARPS * i;
            if (t >= p.R) break;                                           // warp-uniform
            const float wt = w[t];
            const float4 v4 = as_f4(vraw[i]);
            a4.x = fmaf(wt, v4.x, a4.x); a4.y = fmaf(wt, v4.y, a4.y);
            a4.z = fmaf(wt, v4.z, a4.z); a4.w = fmaf(wt, v4.w, a4.w);
            dw += wt;
        }
        *reinterpret_cast<float4 *>(&vacc_sm[warp][4 * lane]) = a4;
        if (lane == 0) vden_sm[warp] = dw;
    }
    // group `grp` takes chunks grp, grp + 4, ...
    float acc = 0.0f, den = 0.0f;
#pragma unroll
    for (int i = 0; i < CB_PART; ++i) {
        const float f = expf(pml[i].x - m);                                // exp(-inf) = 0 for the slots past the last chunk
        acc = fmaf(f, pr[i], acc);
        den = fmaf(f, pml[i].y, den);
    }
    for (int sidx = grp + CB_GROUPS * CB_PART; sidx < p.nchunk; sidx += CB_GROUPS) {
        const float f = expf(ml[2 * sidx] - m);
        acc = fmaf(f, part[(long long)sidx * D + c], acc);
        den = fmaf(f, ml[2 * sidx + 1], den);
    }
    __syncthreads();                                                       // the warps' residual sums are in shared memory
    if (grp == 0) {
#pragma unroll
        for (int wi = 0; wi < CB_WARPS; ++wi) { acc += vacc_sm[wi][c]; if (c == 0) den += vden_sm[wi]; }
    }
    acc_sm[grp][c] = acc;
    if (c == 0) den_sm[grp] = den;
    __syncthreads();
    if (grp == 0) {
        float a = acc_sm[0][c], dsum = den_sm[0];
#pragma unroll
        for (int g = 1; g < CB_GROUPS; ++g) { a += acc_sm[g][c]; dsum += den_sm[g]; }
        p.out[((long long)b * p.Hq + hq) * D + c] = a / dsum;
    }
}

template <int BITS, int NQ, bool ROPE, bool M16>
int launch_partial_r(const AttnParams &p, int qpasses, cudaStream_t st)
{
    const size_t smem = sizeof(float) * (NQ * D + AT_WARPS * NQ * D + NQ * AT_CHUNK + NQ * AT_WARPS + 8) +
                        (ROPE ? sizeof(float2) * 64 * 32 + sizeof(float4) * AT_WARPS * 64 : 0);
    SQUAT_CUDA(cudaFuncSetAttribute(attn_partial_kernel<BITS, NQ, ROPE, M16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    attn_partial_kernel<BITS, NQ, ROPE, M16><<<dim3(p.nchunk * qpasses, p.H, p.B), AT_THREADS, smem, st>>>(p);
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return SQUAT_OK;
}
template <int BITS, int NQ>
int launch_partial(const AttnParams &p, int qpasses, cudaStream_t st)
{
    if (p.meta16) return p.rope_a ? launch_partial_r<BITS, NQ, true, true>(p, qpasses, st) : launch_partial_r<BITS, NQ, false, true>(p, qpasses, st);
    return p.rope_a ? launch_partial_r<BITS, NQ, true, false>(p, qpasses, st) : launch_partial_r<BITS, NQ, false, false>(p, qpasses, st);
}

}  // namespace

size_t squat_attention_workspace_floats(int batch, int n_q_heads, int n_tokens)
{
    const long long nchunk = (n_tokens + 255) / 256;             // the smallest chunk the launcher may choose
    return (size_t)batch * n_q_heads * nchunk * (D + 2);
}

int squat_launch_decode_attention(const void *q, int q_dtype, int batch, int Hq, int H, int T,
                                  const unsigned char *kc, const void *ks, const void *kz,
                                  const unsigned char *vc, const void *vs, const void *vz,
                                  long long csb, long long csh, int bits, int G,
                                  const void *k_res, const void *v_res, int res_dtype, int R,
                                  float scale, float *out, float *workspace,
                                  const float *rope_table, int rope_blocks, long long first_pos, int meta16, cudaStream_t st)
{
    AttnParams p;
    p.meta16 = meta16;
    p.rope_a = reinterpret_cast<const float2 *>(rope_table);                     // NULL: keys were stored after the embedding
    p.rope_b = p.rope_a ? p.rope_a + (size_t)rope_blocks * 64 : nullptr;
    p.first_pos = first_pos;
    p.q = q; p.q_bf16 = q_dtype == SQUAT_BF16; p.B = batch; p.Hq = Hq; p.H = H; p.T = T;
    p.kc = kc; p.vc = vc; p.ks = ks; p.kz = kz; p.vs = vs; p.vz = vz; p.csb = csb; p.csh = csh; p.G = G;
    p.k_res = k_res; p.v_res = v_res; p.res_bf16 = res_dtype == SQUAT_BF16; p.R = R;
    p.scale = scale; p.out = out;
    int sms = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    p.chunk = AT_CHUNK;                                          // smaller chunks while that leaves fewer than ~4 CTAs per SM
    while (p.chunk > 256 && (long long)batch * H * ((T + p.chunk - 1) / p.chunk) < 4LL * sms) p.chunk /= 2;
    p.nchunk = (T + p.chunk - 1) / p.chunk;
    p.part = workspace;
    p.ml = workspace + (size_t)batch * Hq * p.nchunk * D;
    const int qpk = Hq / H;
    if (p.nchunk > 0) {
        int rc;
        if (qpk == 1) rc = bits == 2 ? launch_partial<2, 1>(p, 1, st) : launch_partial<4, 1>(p, 1, st);
        else if (qpk == 2) rc = bits == 2 ? launch_partial<2, 2>(p, 1, st) : launch_partial<4, 2>(p, 1, st);
        else rc = bits == 2 ? launch_partial<2, 4>(p, (qpk + 3) / 4, st) : launch_partial<4, 4>(p, (qpk + 3) / 4, st);
        if (rc != SQUAT_OK) return rc;
    }
    if (p.res_bf16) attn_combine_kernel<true><<<dim3(Hq, batch), CB_THREADS, 0, st>>>(p);
    else attn_combine_kernel<false><<<dim3(Hq, batch), CB_THREADS, 0, st>>>(p);
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return SQUAT_OK;
}
