// Key quantization with error feedback: Algorithm 1, function Quant, with the update of
// Eq. (3) / Eq. (update_block) applied through the assembled matrix W (W[j'][j] multiplies the
// rounding error of channel j into channel j' > j), and the quantizer of Section 2.
//
// Mapping.  A group is G consecutive tokens of one (batch, head); its channels must be visited in
// order, and each channel's grid needs min/max over the group's tokens.  So: lane = token, one warp
// (G = 32) or a team of G/32 warps per group.  The 128 channels are processed in 4 blocks of 32.
//
//   sequential sweep of a block (CUDA cores; 32 channels, unrolled so every register index is static):
//       m, M  = warp min / max (redux.sync on f32)         -> scale = (M-m)/L, zero = m
//       c     = rint((x_j - m)/scale), decided exactly through the remainder c*scale - (x_j - m)
//       e     = fma(c, scale, -(x_j - m))                   (= deq(qtz(x_j)) - x_j)
//       x_j' += e * W[j'][j]  for the later channels j' of the block (the diagonal 32 x 32 block of W^T,
//       read from shared memory as broadcast 16-byte loads, applied with packed fma.rn.f32x2)
//
//   update of the later blocks (tcgen05 tensor cores): three quarters of the multiply-adds are the
//   dense contractions (tokens x 32 errors) x (32 x later channels).  A tile is 128 tokens' worth of
//   groups worked by 4 warps: row m of the tile = lane (m % 32) of the warp with warp % 4 == m / 32 =
//   tensor-memory lane m.  Tensor memory holds, per tile, the fp32 accumulator D[128 x 96] of the
//   corrections to channels 32 .. 127 and, in the tile's other 32 columns, E_hi of the block just swept:
//   the raw fp32 errors (the tensor core reads the top 19 bits of a word: tf32 by truncation).
//   E_lo = e - trunc(e), exact in fp32, goes to shared memory as an A operand (K-major 8 x 16-byte core
//   matrices).  After the sweep of block b the last of the tile's 4 warps to get there issues
//        D[:, 32 b .. 95] (+)= E_lo * Whi_b + E_hi * Wlo_b + E_hi * Whi_b     (12 MMAs of 128 x (96 - 32 b) x 8)
//   with W^T's off-diagonal panels split into tf32 hi / lo (small terms first within a block: the
//   accumulator truncates on every add) and commits them to the tile's mbarrier; nobody waits at a CTA
//   or tile barrier.  Before the next sweep each warp waits for that phase (bounded), reads its 32
//   columns of D with tcgen05.ld -- one token per lane, no transpose -- and adds the keys.
//
// Per head the kernel needs 64 KB in shared memory: the four diagonal blocks (fp32) and the three
// hi / lo panels, copied as they are (cp.async.bulk, counted on an mbarrier) from the image that
// pack_w_kernel writes when the update matrices are built or imported.  Two images fit (head h in buffer
// h & 1).  CTAs are persistent: each takes a contiguous range of tiles and works it in rounds of up to 4
// tiles, one per tile slot, sized as evenly as the range allows; a round may cross one head boundary.
//
// Work per key vector: 8128 fp32 multiply-adds (dense triangle, g = 1): 1984 on the CUDA cores
// (sweeps: four triangles of 32 * 31 / 2), 6144 x 3 tf32 products on the tensor cores.
#include "squat_internal.cuh"
#include <cuda_fp16.h>

namespace {

constexpr int D = SQUAT_D;
constexpr int BLK = 32;                   // channels per block
constexpr int NBLK = D / BLK;             // 4
constexpr float kMagic = 12582912.0f;     // 1.5 * 2^23

constexpr int TC_SLOTS = 4;                          // 128-token tiles in flight per CTA
constexpr int TC_WARPS = TC_SLOTS * 4;
constexpr int TC_THREADS = TC_WARPS * 32;
constexpr int TC_COLS_PER_TILE = 128;                // [0, 96) D: corrections of channels 32 .. 127; [96, 128) E_hi of the block just swept
constexpr int TC_EHI_COL = 96;
constexpr int TC_TMEM_COLS = 512;
static_assert(TC_SLOTS * TC_COLS_PER_TILE <= TC_TMEM_COLS, "tensor memory has 512 columns");
constexpr int TC_E_FLOATS = 128 * BLK;               // one tile's E_hi (or E_lo): 128 rows x 32 channels
constexpr int TC_DIAG_FLOATS = NBLK * BLK * BLK;     // four 32 x 32 diagonal blocks of W^T
constexpr int TC_PANEL_FLOATS = BLK * (3 * BLK + 2 * BLK + BLK);     // panels of source blocks 0..2: (96 - 32 b) x 32
constexpr int TC_IMG_FLOATS = TC_DIAG_FLOATS + 2 * TC_PANEL_FLOATS;  // = d * d: diag | hi panels | lo panels
static_assert(TC_IMG_FLOATS == D * D, "the staged image of W has the size of W");
constexpr unsigned TC_A_LBO = 128 * 16, TC_SBO = 128;                 // bytes
__host__ __device__ constexpr int tc_panel_off(int b) { return b == 0 ? 0 : (b == 1 ? 3 * BLK * BLK : 5 * BLK * BLK); }
// instruction descriptor: fp32 accumulator, tf32 A and B, both K-major, N = n, M = 128
__host__ __device__ constexpr unsigned tc_idesc(int n) { return (1u << 4) | (2u << 7) | (2u << 10) | ((unsigned)(n >> 3) << 17) | ((128u >> 4) << 24); }

typedef unsigned long long u64;

__device__ __forceinline__ u64 pack2(float lo, float hi)
{
    u64 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ float lo_of(u64 v)
{
    return __uint_as_float((unsigned)(v & 0xffffffffull));
}
__device__ __forceinline__ float hi_of(u64 v)
{
    return __uint_as_float((unsigned)(v >> 32));
}
__device__ __forceinline__ u64 ffma2(u64 a, u64 b, u64 c)
{
    u64 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
// Warp-wide min / max.  The NaN-propagating forms: a NaN key makes the group's grid NaN, which the check of the stored
// scale reports (SQUAT_FLAG_NONFINITE), instead of vanishing in the reduction and corrupting the codes unnoticed.
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

// ---- tcgen05 / tensor-memory helpers (5th-generation tensor cores) -------------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void *ptr) { return (unsigned)__cvta_generic_to_shared(ptr); }
__device__ __forceinline__ unsigned tf32_of(float x)             // round to nearest tf32 (10 mantissa bits)
{
    unsigned r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return r;
}
// 32 consecutive columns of the warp's lanes into registers (lane l gets row l)
__device__ __forceinline__ void tmem_ld32(unsigned taddr, unsigned (&r)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// shared-memory matrix descriptor, no swizzle, K-major: 8 x 16-byte core matrices, lbo bytes between the two
// halves of a K step, sbo bytes between groups of 8 rows
__device__ __forceinline__ u64 umma_desc(unsigned addr, unsigned lbo, unsigned sbo)
{
    return (u64)((addr & 0x3FFFF) >> 4) | ((u64)(lbo >> 4) << 16) | ((u64)(sbo >> 4) << 32) | (1ull << 46);
}
// D[128 x N] (+)= A[128 x 8] * B[N x 8]^T, tf32 operands from shared memory, fp32 accumulation in tensor memory
__device__ __forceinline__ void umma_tf32_ss(unsigned d_taddr, u64 a_desc, u64 b_desc, unsigned idesc, unsigned accumulate)
{
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                 " tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d_taddr), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// the same with A from tensor memory (rows = lanes, 8 consecutive 32-bit columns)
__device__ __forceinline__ void umma_tf32_ts(unsigned d_taddr, unsigned a_taddr, u64 b_desc, unsigned idesc, unsigned accumulate)
{
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                 " tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n}"
                 ::"r"(d_taddr), "r"(a_taddr), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// 4 consecutive 32-bit columns of the warp's 32 tensor-memory lanes: lane l writes its own row
__device__ __forceinline__ void tmem_st4(unsigned taddr, float a, float b, float c, float d)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1, %2, %3, %4};"
                 ::"r"(taddr), "r"(__float_as_uint(a)), "r"(__float_as_uint(b)), "r"(__float_as_uint(c)), "r"(__float_as_uint(d)) : "memory");
}
__device__ __forceinline__ void umma_commit(unsigned mbar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(mbar) : "memory");
}
// Bounded wait for a phase of an mbarrier: false when the limit ran out (the caller records it and moves on).
__device__ __forceinline__ bool mbar_wait(unsigned mbar, unsigned parity)
{
    for (int it = 0; it < (1 << 22); ++it) {
        unsigned done;
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                     : "=r"(done) : "r"(mbar), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}

// Starts the copy of one head's 64 KB image into shared memory on the bulk-copy engine (one CTA, one destination); the bytes are
// counted on `mbar`, whose current phase completes when all of them have landed.
__device__ __forceinline__ void stage_image_async(float *dst, const float *src, unsigned mbar)
{
    constexpr unsigned BYTES = TC_IMG_FLOATS * 4, PIECE = 16384;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // earlier reads of the old image, before the engine's writes
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar), "r"(BYTES) : "memory");
#pragma unroll
    for (unsigned o = 0; o < BYTES; o += PIECE)
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_u32(dst) + o), "l"(reinterpret_cast<const char *>(src) + o), "r"(PIECE), "r"(mbar) : "memory");
}

struct KeyParams {
    const float *Wimg;        // [H, d * d] staged images of the update matrices (pack_w_kernel)
    const void *k;
    long long sb, sh, st;     // element strides of k
    unsigned char *codes;
    void *scales, *zeros;     // float32, or binary16 in the M16 instances
    long long osb, osh;       // output strides in tokens
    int B, H, T;
    int groups_per_bh;        // T / G
    int groups_per_head;      // B * T / G
    int tiles_per_head;       // 128-token tiles per head (the last one may be ragged)
    int total_tiles;          // H * tiles_per_head
    unsigned *status;
    const int *exact_blocks;  // device word: leading 32-channel blocks that no earlier channel corrects (see sweep_block)
#ifdef SQUAT_CHECKED
    SqExtent x_k, x_codes, x_scales, x_zeros, x_img;      // what the caller's tensors and the handle's images span
#endif
};

// What the sweep may touch, for the bounds-checked build (empty otherwise).
struct SweepChk {
#ifdef SQUAT_CHECKED
    unsigned *status;
    const float *img;         // the staged image the diagonal block belongs to
    const float *e_region;    // the tile slot's E_lo operand
    unsigned tmem_lo, tmem_hi;   // the columns of the tile's E_hi operand: [lo, hi)
#endif
};

template <bool BF16>
struct RawRow {
    uint4 v[BF16 ? 4 : 8];      // 32 channels of one token
};
template <bool BF16>
__device__ __forceinline__ void load_row(RawRow<BF16> &r, const void *row, int chan)
{
    if (BF16) {
        const uint4 *q = reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(row) + chan);
#pragma unroll
        for (int i = 0; i < 4; ++i) r.v[i] = __ldg(q + i);
    } else {
        const uint4 *q = reinterpret_cast<const uint4 *>(reinterpret_cast<const float *>(row) + chan);
#pragma unroll
        for (int i = 0; i < 8; ++i) r.v[i] = __ldg(q + i);
    }
}
// channel pair q (channels 2q, 2q + 1) of the row as two floats
template <bool BF16>
__device__ __forceinline__ float2 row_pair(const RawRow<BF16> &r, int q)
{
    if (BF16) {
        const uint4 &t = r.v[q >> 2];
        const unsigned w = (q & 3) == 0 ? t.x : (q & 3) == 1 ? t.y : (q & 3) == 2 ? t.z : t.w;
        return make_float2(bf16lo_to_f32(w), bf16hi_to_f32(w));
    } else {
        const uint4 &t = r.v[q >> 1];
        return (q & 1) ? make_float2(__uint_as_float(t.z), __uint_as_float(t.w))
                       : make_float2(__uint_as_float(t.x), __uint_as_float(t.y));
    }
}

// The sequential part: the 32 channels of one block, one token per lane, values in xp (16 packed pairs).
// For every channel: grid from the warp (team) min / max, rounding decision, error e; e is pushed onto the
// later channels of the block through the diagonal 32 x 32 block of W^T and written, 4 channels at a time, to
// this lane's row of the tile's A operands (e_hi, e_lo: 4 floats per 4-channel chunk, chunks TC_A_LBO bytes
// apart) for the tensor-core update of the later blocks.
//
// Rounding decision.  t = (x - m) / scale is formed as (x - m) * L * rcp(M - m) with the hardware reciprocal,
// so c0 = rint(t) can be off by one when t is within ~1e-6 of a rounding midpoint.  Channels that earlier
// channels have corrected hold generic float32 values and such near-ties are as rare as that bound; but
// channels nothing has corrected yet (the first g channels, or all of them when W = 0) hold raw bf16 / f32
// inputs, where exact ties are structural (x exactly half way between min and max).  For those blocks
// (EXACT) the remainder e0 = c0*scale - (x - m), which is exact next to a midpoint, is compared with
// +-scale/2: that settles the rounding exactly as real arithmetic on the stored float32 scale would, ties
// going to the even code (the threshold of an odd c0 is one ulp lower, so "remainder == scale/2" moves it).
//
// M16: scale and zero-point are stored as binary16.  The float32 values are rounded once more, and the decision
// and the error fed back are taken against the rounded (stored) values: t = (x - z16) / s16, clamped to [0, L]
// because z16 can lie above the group's minimum.
template <int BITS, int NW, bool EXACT, bool M16>
__device__ __forceinline__ void sweep_block(u64 (&xp)[BLK / 2], const float *diag, unsigned e_hi_taddr, float *e_lo, bool store_e,
                                            int lane, int bar_id, int wteam, float2 *red,
                                            uint32_t (&cw)[BLK * BITS / 32], float &my_scale, float &my_zero, const SweepChk &ck)
{
    constexpr float L = float((1 << BITS) - 1);
    constexpr int PER_ACC = 16 / BITS;              // codes accumulated exactly in one float (16 bits of mantissa)
    float cacc[BLK / PER_ACC];
    float eh[4], el[4];
#pragma unroll
    for (int jj = 0; jj < BLK; ++jj) {
        const float xj = (jj & 1) ? hi_of(xp[jj >> 1]) : lo_of(xp[jj >> 1]);
        float m = warp_min(xj);
        float Mx = warp_max(xj);
        if (NW > 1) {
            float2 *slot = red + (jj & 1) * NW;             // [parity][warp of the team]
            (void)ck;
            if (lane == 0) slot[wteam] = make_float2(m, Mx);
            team_barrier(bar_id, 32 * NW);
#pragma unroll
            for (int w = 0; w < NW; ++w) {
                const float2 o = slot[w];
                m = min_nan(m, o.x);
                Mx = max_nan(Mx, o.y);
            }
        }
        const float rng = __fsub_rn(Mx, m);
        // the stored scale: the correctly rounded quotient where the block's decisions are exact (raw inputs: bit-identical to
        // plain round-to-nearest quantization), else the product with RN(1/L) (within one ulp of it; one instruction, not three)
        float scale = EXACT ? div_by_levels<BITS>(rng) : __fmul_rn(rng, 1.0f / L);
        float rcp, y0, dlt;
        if (M16) {
            scale = __half2float(__float2half_rn(scale));
            m = __half2float(__float2half_rn(m));
            dlt = __fsub_rn(xj, m);
            asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(rcp) : "f"(scale));
            rcp = scale > 0.0f ? rcp : 0.0f;                                       // scale 0 (no range, or underflow): codes 0
            y0 = __fmaf_rn(dlt, rcp, kMagic);
        } else {
            dlt = __fsub_rn(xj, m);
            const float dltL = __fmul_rn(dlt, L);
            asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(rcp) : "f"(fmaxf(rng, 1e-30f)));   // constant group: dlt = 0 -> code 0
            y0 = __fmaf_rn(dltL, rcp, kMagic);
        }
        float c = __fsub_rn(y0, kMagic);
        float e = __fmaf_rn(c, scale, -dlt);
        if (EXACT) {
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
        // pack the code arithmetically: sum of c * 2^(BITS k) is exact in float32 up to 16 bits
        if (jj % PER_ACC == 0) cacc[jj / PER_ACC] = c;
        else cacc[jj / PER_ACC] = __fmaf_rn(c, float(1 << ((jj % PER_ACC) * BITS)), cacc[jj / PER_ACC]);
        if (lane == jj) {                               // lane jj keeps channel jj's grid for the store after the sweep
            my_scale = scale;
            my_zero = m;
        }
        // tf32 split by truncation: the tensor core reads only the top 19 bits of each word, so e itself serves
        // as E_hi = trunc(e), and E_lo = e - trunc(e) is exact in fp32
        eh[jj & 3] = e;
        el[jj & 3] = __fsub_rn(e, __uint_as_float(__float_as_uint(e) & 0xffffe000u));
        if ((jj & 3) == 3 && store_e) {
#ifdef SQUAT_CHECKED
            const unsigned col = (e_hi_taddr + (jj - 3)) & 0xffffu;
            const bool ok_t = sq_chk(col >= ck.tmem_lo && col + 4 <= ck.tmem_hi, ck.status);
            const bool ok_s = sq_chk(sq_inside(e_lo + (jj >> 2) * (TC_A_LBO / 4), 16, ck.e_region, TC_E_FLOATS * 4), ck.status);
            if (ok_t) tmem_st4(e_hi_taddr + (jj - 3), eh[0], eh[1], eh[2], eh[3]);
            if (ok_s) *reinterpret_cast<float4 *>(e_lo + (jj >> 2) * (TC_A_LBO / 4)) = make_float4(el[0], el[1], el[2], el[3]);
#else
            tmem_st4(e_hi_taddr + (jj - 3), eh[0], eh[1], eh[2], eh[3]);
            *reinterpret_cast<float4 *>(e_lo + (jj >> 2) * (TC_A_LBO / 4)) = make_float4(el[0], el[1], el[2], el[3]);
#endif
        }
        const u64 ee = pack2(e, e);
        const float *wrow = diag + jj * BLK;
#ifdef SQUAT_CHECKED
        if (!sq_chk(sq_inside(wrow, BLK * 4, ck.img, TC_DIAG_FLOATS * 4), ck.status)) continue;    // the reads below stay inside this row
#endif
        // later channels of the block, 4 per 16-byte broadcast read; where only the upper half of the first chunk
        // is still to come, an 8-byte read does (a broadcast read is charged by its width)
        if ((jj + 1) % 4 >= 2) {
            const int q = (jj + 1) / 4;
            const u64 wy = *reinterpret_cast<const u64 *>(wrow + 4 * q + 2);
            xp[2 * q + 1] = ffma2(ee, wy, xp[2 * q + 1]);
        }
#pragma unroll
        for (int q = ((jj + 1) % 4 >= 2 ? (jj + 1) / 4 + 1 : (jj + 1) / 4); q < BLK / 4; ++q) {
            const ulonglong2 wv = *reinterpret_cast<const ulonglong2 *>(wrow + 4 * q);
            if (2 * q >= (jj + 1) / 2) xp[2 * q] = ffma2(ee, wv.x, xp[2 * q]);
            xp[2 * q + 1] = ffma2(ee, wv.y, xp[2 * q + 1]);
        }
    }
#pragma unroll
    for (int w = 0; w < BLK * BITS / 32; ++w)
        cw[w] = (uint32_t)__float2int_rn(cacc[2 * w]) | ((uint32_t)__float2int_rn(cacc[2 * w + 1]) << 16);
}

// Where one warp's 32 tokens of a round come from and go to.
struct TileRows {
    bool active;              // the warp's group exists (a head's last tile may be ragged: its spare warps redo the last
                              // group and store nothing)
    int head;
    const void *row;          // this lane's key vector
    unsigned char *codes;     // this lane's code row
    long long meta;           // offset of the group's scales / zeros (lane = channel within a block)
};

template <int BITS, int NW, bool BF16, bool M16>
__global__ void __launch_bounds__(TC_THREADS, 1) quant_keys_kernel(const KeyParams p)
{
    constexpr int G = 32 * NW;
    constexpr int GPT = 4 / NW;                          // groups per tile
    constexpr int NTEAMS = TC_SLOTS * GPT;               // teams of NW warps
    constexpr int WORDS_PER_BLK = BLK * BITS / 32;       // 2 (2-bit) or 4 (4-bit)
    extern __shared__ __align__(128) float smem[];
    float *Eall = smem;                                  // [TC_SLOTS][TC_E_FLOATS]: the tiles' E_lo operands
    float *images = Eall + TC_SLOTS * TC_E_FLOATS;       // [2][TC_IMG_FLOATS]: head h's image lives in buffer h & 1
    float2 *red_all = reinterpret_cast<float2 *>(images + 2 * TC_IMG_FLOATS);    // [NTEAMS][2][NW]
    u64 *mbar = reinterpret_cast<u64 *>(red_all + NTEAMS * 2 * NW);              // [TC_SLOTS] MMAs done, [1] image staged
    // [0] tensor-memory base, [1] a bounded wait ran out, [2 + slot] arrivals of the slot's warps, [2 + TC_SLOTS] the
    // number of leading blocks that take the exact rounding decision (read once from the handle's device word)
    volatile unsigned *shared_words = reinterpret_cast<volatile unsigned *>(mbar + TC_SLOTS + 1);

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int slot = warp >> 2;                          // tile slot of this warp
    const int wq = warp & 3;                             // its quarter of the tile = its tensor-memory lanes
    const int team = slot * GPT + wq / NW;
    const int wteam = wq % NW;
    float2 *red = red_all + team * (2 * NW);

    // A CTA takes a contiguous range of tiles (head-major order) and works it in rounds of up to TC_SLOTS tiles, one per
    // slot, sized as evenly as its range allows (7 tiles = 4 + 3, not 4 + 4 elsewhere).  Two images fit in shared memory,
    // so a round may run across one head boundary.  (All of this in 32-bit integers and recomputed rather than kept:
    // the sweeps need every register.)
    const int t_lo = (int)((long long)p.total_tiles * blockIdx.x / gridDim.x);
    const int t_hi = (int)((long long)p.total_tiles * (blockIdx.x + 1) / gridDim.x);
    auto round_size = [&](int start) {
        const int left = t_hi - start;
        if (left <= 0) return 0;
        const int rounds_left = (left + TC_SLOTS - 1) / TC_SLOTS;
        int n = (left + rounds_left - 1) / rounds_left;
        const int two_heads_end = (start / p.tiles_per_head + 2) * p.tiles_per_head;
        if (n > two_heads_end - start) n = two_heads_end - start;
        return n;
    };
    const unsigned img_mbar = smem_u32(mbar + TC_SLOTS);
    unsigned img_phase = 0;

    if (threadIdx.x == 32) {
#pragma unroll
        for (int t = 0; t < TC_SLOTS; ++t) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(mbar + t)), "r"(1) : "memory");
            shared_words[2 + t] = 0;
        }
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(img_mbar), "r"(1) : "memory");
        shared_words[1] = 0;
        shared_words[2 + TC_SLOTS] = (unsigned)__ldg(p.exact_blocks);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // the first head's image is on its way while the rest of the set-up runs
        if (t_lo < t_hi) {
            const int h0 = t_lo / p.tiles_per_head;
            if (SQ_CHK_G(p.status, p.Wimg + (long long)h0 * TC_IMG_FLOATS, TC_IMG_FLOATS * 4, p.x_img))
            stage_image_async(images + (h0 & 1) * TC_IMG_FLOATS, p.Wimg + (long long)h0 * TC_IMG_FLOATS, img_mbar);
        }
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(const_cast<unsigned *>(shared_words))), "r"((unsigned)TC_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_base = shared_words[0];
    const unsigned t_tile = tmem_base + slot * TC_COLS_PER_TILE;               // lane field 0: the MMAs' accumulator
    const unsigned t_mine = t_tile + ((unsigned)(wq * 32) << 16);              // this warp's 32 lanes
    float *e_lo = Eall + slot * TC_E_FLOATS + (wq * 32 + lane) * 4;            // this lane's row of the tile's E_lo operand
    const unsigned a_lo = smem_u32(Eall + slot * TC_E_FLOATS);
    const unsigned my_mbar = smem_u32(mbar + slot);
    unsigned phase = 0;

    auto locate = [&](int tile, TileRows &t) {
        const int h = tile / p.tiles_per_head;
        const int g_raw = (tile - h * p.tiles_per_head) * GPT + wq / NW;                  // group within the head
        t.head = h;
        t.active = g_raw < p.groups_per_head;
        const int in_head = t.active ? g_raw : p.groups_per_head - 1;
        const int b = in_head / p.groups_per_bh;
        const int grp = in_head - b * p.groups_per_bh;
        const int tok = grp * G + wteam * 32 + lane;
        const long long out_tok0 = (long long)b * p.osb + (long long)h * p.osh;
        t.codes = p.codes + (out_tok0 + tok) * (D * BITS / 8);
        t.meta = (out_tok0 / G + grp) * D + lane;
        const long long row_off = (long long)b * p.sb + (long long)h * p.sh + (long long)tok * p.st;
        t.row = BF16 ? static_cast<const void *>(reinterpret_cast<const __nv_bfloat16 *>(p.k) + row_off)
                     : static_cast<const void *>(reinterpret_cast<const float *>(p.k) + row_off);
    };

    // every read of a key row goes through here (the bounds-checked build tests the 32 channels' bytes against the tensor)
    auto load_keys = [&](RawRow<BF16> &r, const void *row, int chan) {
        if (SQ_CHK_G(p.status, static_cast<const char *>(row) + chan * (BF16 ? 2 : 4), BLK * (BF16 ? 2 : 4), p.x_k))
            load_row<BF16>(r, row, chan);
    };
    RawRow<BF16> raw;
    int start = t_lo;
    if (slot < round_size(start)) {
        TileRows first;
        locate(start + slot, first);
        load_keys(raw, first.row, 0);                    // in flight while the first head is staged
    }
    int max_staged = -1;     // heads come in increasing order: the buffers hold max_staged and, earlier, max_staged - 1
    while (start < t_hi) {
        const int n_round = round_size(start);
        // images of the (at most two) heads of this round
        const int h_first = start / p.tiles_per_head, h_last = (start + n_round - 1) / p.tiles_per_head;
        for (int hh = h_first; hh <= h_last; ++hh) {
            if (hh <= max_staged) continue;
            if (max_staged >= 0) {                       // (the very first copy was started at kernel entry)
                __syncthreads();                         // every read of the buffer's old image, by a lane or by an MMA, is over
                if (threadIdx.x == 32 && SQ_CHK_G(p.status, p.Wimg + (long long)hh * TC_IMG_FLOATS, TC_IMG_FLOATS * 4, p.x_img))
                    stage_image_async(images + (hh & 1) * TC_IMG_FLOATS, p.Wimg + (long long)hh * TC_IMG_FLOATS, img_mbar);
            }
            if (!shared_words[1] && !mbar_wait(img_mbar, img_phase)) {   // bounded, like every wait here
                shared_words[1] = 1;
                atomicOr(p.status, SQUAT_FLAG_DEVICE_TIMEOUT);
            }
            img_phase ^= 1;
            max_staged = hh;
        }
        const bool valid = slot < n_round;
        const bool nxt_valid = slot < round_size(start + n_round);
        const void *nxt_row = nullptr;
        if (nxt_valid) {
            TileRows nxt;
            locate(start + n_round + slot, nxt);
            nxt_row = nxt.row;
        }
        TileRows cur;
        cur.head = 0;
        if (valid) locate(start + slot, cur);

        const float *img = images + (cur.head & 1) * TC_IMG_FLOATS;       // diagonal blocks | hi panels | lo panels
        const float *Bhi = img + TC_DIAG_FLOATS, *Blo = Bhi + TC_PANEL_FLOATS;
        if (valid) {
#pragma unroll 1
            for (int blk = 0; blk < NBLK; ++blk) {
                u64 xp[BLK / 2];
                if (blk == 0) {
#pragma unroll
                    for (int q = 0; q < BLK / 2; ++q) {
                        const float2 kv = row_pair<BF16>(raw, q);
                        xp[q] = pack2(kv.x, kv.y);
                    }
                } else {
                    // the MMAs that complete this block's corrections were committed after the previous sweep
                    if (!shared_words[1] && !mbar_wait(my_mbar, phase)) {
                        shared_words[1] = 1;
                        atomicOr(p.status, SQUAT_FLAG_DEVICE_TIMEOUT);
                    }
                    phase ^= 1;
                    tc_fence_after();
                    unsigned dv[32];
#ifdef SQUAT_CHECKED
                    {
                        const unsigned col = (t_mine + (blk - 1) * BLK) & 0xffffu, lo = t_tile & 0xffffu;
                        if (!sq_chk(col >= lo && col + 32 <= lo + TC_EHI_COL && ((t_mine >> 16) & 0x7f) == (unsigned)(wq * 32) &&
                                    lo + TC_COLS_PER_TILE <= (tmem_base & 0xffffu) + TC_TMEM_COLS, p.status)) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) dv[i] = 0;
                        } else
                            tmem_ld32(t_mine + (blk - 1) * BLK, dv);
                    }
#else
                    tmem_ld32(t_mine + (blk - 1) * BLK, dv);
#endif
#pragma unroll
                    for (int q = 0; q < BLK / 2; ++q) {
                        const float2 kv = row_pair<BF16>(raw, q);
                        xp[q] = pack2(__fadd_rn(kv.x, __uint_as_float(dv[2 * q])), __fadd_rn(kv.y, __uint_as_float(dv[2 * q + 1])));
                    }
                }
                const bool more = blk + 1 < NBLK;
                // prefetch: the next block of this tile, or the first block of the next round's tile
                if (more) load_keys(raw, cur.row, (blk + 1) * BLK);
                else if (nxt_valid) load_keys(raw, nxt_row, 0);

                const float *diag = img + blk * BLK * BLK;
                uint32_t cw[WORDS_PER_BLK];
                float my_scale = 0.0f, my_zero = 0.0f;
                SweepChk ck;
#ifdef SQUAT_CHECKED
                ck.status = p.status;
                ck.img = img;
                ck.e_region = Eall + slot * TC_E_FLOATS;
                ck.tmem_lo = (t_tile & 0xffffu) + TC_EHI_COL;
                ck.tmem_hi = (t_tile & 0xffffu) + TC_COLS_PER_TILE;
#endif
                if (blk < (int)shared_words[2 + TC_SLOTS])
                    sweep_block<BITS, NW, true, M16>(xp, diag, t_mine + TC_EHI_COL, e_lo, more, lane, 1 + team, wteam, red, cw, my_scale, my_zero, ck);
                else
                    sweep_block<BITS, NW, false, M16>(xp, diag, t_mine + TC_EHI_COL, e_lo, more, lane, 1 + team, wteam, red, cw, my_scale, my_zero, ck);

                if (more) {
                    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");   // E_hi is in tensor memory
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // E_lo rows, for the tensor core
                    tc_fence_before();
                    __threadfence_block();
                    __syncwarp();
                    // the last of the slot's four warps to get here issues the MMAs; nobody waits at a barrier
                    bool last = false;
                    if (lane == 0) last = (atomicAdd(const_cast<unsigned *>(shared_words) + 2 + slot, 1u) & 3u) == 3u;
                    if (last) {
                        __threadfence_block();
                        tc_fence_after();
                        const int nb = 3 * BLK - blk * BLK;        // channels still to come: 96, 64, 32
                        const unsigned idesc = tc_idesc(nb);
                        const unsigned b_lbo = 16u * nb;
                        const unsigned bhi = smem_u32(Bhi + tc_panel_off(blk)), blo = smem_u32(Blo + tc_panel_off(blk));
                        const unsigned d = t_tile + blk * BLK;
#ifdef SQUAT_CHECKED
                        // the windows the descriptors open: A = this slot's E_lo operand, B = the panels of source block blk
                        // inside the staged image, D / A-from-tensor-memory = columns of this tile
                        const unsigned img_lo = smem_u32(img), e_lo_lo = smem_u32(Eall + slot * TC_E_FLOATS);
                        const unsigned panel_bytes = (unsigned)nb * BLK * 4;
                        const bool desc_ok =
                            a_lo == e_lo_lo && a_lo + (BLK / 8 - 1) * 2 * TC_A_LBO + 2 * TC_A_LBO <= e_lo_lo + TC_E_FLOATS * 4 &&
                            bhi >= img_lo + TC_DIAG_FLOATS * 4 && bhi + panel_bytes <= img_lo + (TC_DIAG_FLOATS + TC_PANEL_FLOATS) * 4 &&
                            blo >= img_lo + (TC_DIAG_FLOATS + TC_PANEL_FLOATS) * 4 && blo + panel_bytes <= img_lo + TC_IMG_FLOATS * 4 &&
                            (a_lo & 15u) == 0 && (bhi & 15u) == 0 && (blo & 15u) == 0 &&
                            (d & 0xffffu) + nb <= (t_tile & 0xffffu) + TC_EHI_COL &&
                            (t_tile & 0xffffu) + TC_COLS_PER_TILE <= (tmem_base & 0xffffu) + TC_TMEM_COLS;
                        if (sq_chk(desc_ok, p.status)) {
#endif
#pragma unroll
                        for (int ks = 0; ks < BLK / 8; ++ks)         // E_lo (shared memory) x Whi
                            umma_tf32_ss(d, umma_desc(a_lo + ks * 2 * TC_A_LBO, TC_A_LBO, TC_SBO),
                                         umma_desc(bhi + ks * 2 * b_lbo, b_lbo, TC_SBO), idesc, (blk | ks) != 0);
#pragma unroll
                        for (int ks = 0; ks < BLK / 8; ++ks)         // E_hi (tensor memory) x Wlo
                            umma_tf32_ts(d, t_tile + TC_EHI_COL + 8 * ks, umma_desc(blo + ks * 2 * b_lbo, b_lbo, TC_SBO), idesc, 1u);
#pragma unroll
                        for (int ks = 0; ks < BLK / 8; ++ks)         // E_hi x Whi
                            umma_tf32_ts(d, t_tile + TC_EHI_COL + 8 * ks, umma_desc(bhi + ks * 2 * b_lbo, b_lbo, TC_SBO), idesc, 1u);
#ifdef SQUAT_CHECKED
                        }
#endif
                        umma_commit(my_mbar);
                    }
                    __syncwarp();
                }

                if (cur.active) {
                    unsigned char *cp = cur.codes + blk * (BLK * BITS / 8);
                    if (!SQ_CHK_G(p.status, cp, BLK * BITS / 8, p.x_codes)) {
                    } else if (WORDS_PER_BLK == 2)
                        *reinterpret_cast<uint2 *>(cp) = make_uint2(cw[0], cw[1]);
                    else
                        *reinterpret_cast<uint4 *>(cp) = make_uint4(cw[0], cw[1], cw[WORDS_PER_BLK > 2 ? 2 : 0], cw[WORDS_PER_BLK > 2 ? 3 : 0]);
                    if (wteam == 0 && SQ_CHK_G(p.status, static_cast<char *>(p.scales) + (cur.meta + blk * BLK) * (M16 ? 2 : 4), M16 ? 2 : 4, p.x_scales) &&
                        SQ_CHK_G(p.status, static_cast<char *>(p.zeros) + (cur.meta + blk * BLK) * (M16 ? 2 : 4), M16 ? 2 : 4, p.x_zeros)) {
                        if (M16) {
                            reinterpret_cast<__half *>(p.scales)[cur.meta + blk * BLK] = __float2half_rn(my_scale);   // exact
                            reinterpret_cast<__half *>(p.zeros)[cur.meta + blk * BLK] = __float2half_rn(my_zero);
                        } else {
                            reinterpret_cast<float *>(p.scales)[cur.meta + blk * BLK] = my_scale;
                            reinterpret_cast<float *>(p.zeros)[cur.meta + blk * BLK] = my_zero;
                        }
                        if (!(my_scale > 0.0f && my_scale < __int_as_float(0x7f800000)))
                            atomicOr(p.status, my_scale == 0.0f ? SQUAT_FLAG_ZERO_RANGE : SQUAT_FLAG_NONFINITE);
                    }
                }
            }
        } else if (nxt_valid) {
            load_keys(raw, nxt_row, 0);
        }
        start += n_round;
    }

    // Every committed batch has been waited for unless a wait ran out; then commit once more per slot and give the
    // tensor core a bounded time to drain before the columns are handed back.
    if (shared_words[1] && wq == 0 && lane == 0) {
        umma_commit(my_mbar);
        mbar_wait(my_mbar, phase);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((unsigned)TC_TMEM_COLS) : "memory");
}

// Writes, per head, the 64 KB image of the update matrix that the key kernel stages in shared memory:
//   [0, 4096)        the four diagonal 32 x 32 blocks of W^T, row-major: block b, row jj, column c = W^T[32 b + jj][32 b + c]
//   [4096, 10240)    hi panels of source blocks b = 0, 1, 2: B_b(n, k) = W[32 (b + 1) + n][32 b + k] = W^T[32 b + k][32 (b + 1) + n],
//                    n < 96 - 32 b, k < 32, rounded to tf32, K-major in 8 x 16-byte core matrices:
//                    float index (k / 4) * 4 N + 4 n + k % 4 with N = 96 - 32 b
//   [10240, 16384)   lo panels: tf32(W - hi), same layout
// PACK_SLICES CTAs per head (grid (heads, slices): the kernel is a chain of two dependent global accesses, so more CTAs,
// not more work per thread, shorten it); each thread takes (panel, 4-k chunk, channel n): four coalesced row reads, one
// 16-byte store.
__global__ void __launch_bounds__(256) pack_w_kernel(const float *__restrict__ Wt, float *__restrict__ Wimg, int exact_blocks,
                                                     int *__restrict__ exact_blocks_dev)
{
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) *exact_blocks_dev = exact_blocks;    // travels with the matrices it describes
    const float *src = Wt + (long long)blockIdx.x * D * D;
    float *img = Wimg + (long long)blockIdx.x * TC_IMG_FLOATS;
    const int first = blockIdx.y * blockDim.x + threadIdx.x, stride = gridDim.y * blockDim.x;
    for (int i = first; i < TC_DIAG_FLOATS / 4; i += stride) {
        const int b = i / (BLK * BLK / 4), r = i % (BLK * BLK / 4), jj = r / (BLK / 4), c4 = r % (BLK / 4);
        reinterpret_cast<float4 *>(img)[i] = __ldg(reinterpret_cast<const float4 *>(src + (b * BLK + jj) * D + b * BLK + 4 * c4));
    }
    float *Bhi = img + TC_DIAG_FLOATS, *Blo = Bhi + TC_PANEL_FLOATS;
    for (int i = first; i < TC_PANEL_FLOATS / 4; i += stride) {
        const int f = 4 * i;                                 // first float of the 16-byte unit
        const int b = f < tc_panel_off(1) ? 0 : (f < tc_panel_off(2) ? 1 : 2);
        const int nb = 3 * BLK - b * BLK;
        const int r = (f - tc_panel_off(b)) / 4;             // unit within the panel: kc * nb + n
        const int kc = r / nb, n = r % nb;
        const float *g = src + (b * BLK + 4 * kc) * D + (b + 1) * BLK + n;
        const float w0 = __ldg(g), w1 = __ldg(g + D), w2 = __ldg(g + 2 * D), w3 = __ldg(g + 3 * D);
        const float4 whi = make_float4(__uint_as_float(tf32_of(w0)), __uint_as_float(tf32_of(w1)),
                                       __uint_as_float(tf32_of(w2)), __uint_as_float(tf32_of(w3)));
        reinterpret_cast<float4 *>(Bhi)[i] = whi;
        reinterpret_cast<float4 *>(Blo)[i] =
            make_float4(__uint_as_float(tf32_of(__fsub_rn(w0, whi.x))), __uint_as_float(tf32_of(__fsub_rn(w1, whi.y))),
                        __uint_as_float(tf32_of(__fsub_rn(w2, whi.z))), __uint_as_float(tf32_of(__fsub_rn(w3, whi.w))));
    }
}

template <int BITS, int NW, bool BF16, bool M16>
int launch_keys_inst(const KeyParams &p, int grid, size_t smem, cudaStream_t st)
{
    SQUAT_CUDA(cudaFuncSetAttribute(quant_keys_kernel<BITS, NW, BF16, M16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    quant_keys_kernel<BITS, NW, BF16, M16><<<grid, TC_THREADS, smem, st>>>(p);
    return SQUAT_OK;
}

template <int BITS, int NW>
int launch_keys(KeyParams p, int dtype, int meta16, cudaStream_t st)
{
    const long long groups_per_head = (long long)p.B * p.groups_per_bh;
    const long long tiles_per_head = (groups_per_head + 4 / NW - 1) / (4 / NW);
    if (tiles_per_head * p.H > 0x7fffffffLL) return SQUAT_ERR_UNSUPPORTED;          // the kernel counts tiles in 32 bits
    p.groups_per_head = (int)groups_per_head;
    p.tiles_per_head = (int)tiles_per_head;
    p.total_tiles = (int)(tiles_per_head * p.H);

    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    constexpr int GPT = 4 / NW;
    constexpr int NTEAMS = TC_SLOTS * GPT;
    // 193 KB: well over half an SM's shared memory, so two CTAs (each asking for all 512 tensor-memory columns)
    // never share an SM
    const size_t smem = sizeof(float) * (TC_SLOTS * TC_E_FLOATS + 2 * TC_IMG_FLOATS) +
                        sizeof(float2) * (NTEAMS * 2 * NW) + sizeof(u64) * (TC_SLOTS + 1) + 4 * (3 + TC_SLOTS) + 8;
    const int grid = p.total_tiles < sms ? p.total_tiles : sms;                     // one tile per CTA at least
    int rc;
    if (dtype == SQUAT_BF16) rc = meta16 ? launch_keys_inst<BITS, NW, true, true>(p, grid, smem, st) : launch_keys_inst<BITS, NW, true, false>(p, grid, smem, st);
    else rc = meta16 ? launch_keys_inst<BITS, NW, false, true>(p, grid, smem, st) : launch_keys_inst<BITS, NW, false, false>(p, grid, smem, st);
    if (rc != SQUAT_OK) return rc;
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return SQUAT_OK;
}

}  // namespace

int squat_launch_pack_update_matrices(const float *Wt, float *Wimg, int H, int exact_blocks, int *exact_blocks_dev, cudaStream_t st)
{
    constexpr int PACK_SLICES = 8;
    pack_w_kernel<<<dim3(H, PACK_SLICES), 256, 0, st>>>(Wt, Wimg, exact_blocks, exact_blocks_dev);
    squat_count_launch();
    SQUAT_LAUNCH_CHECK();
    return SQUAT_OK;
}

int squat_launch_quant_keys(const float *Wimg, const void *k, int dtype, int batch, int H, int T,
                            long long sb, long long sh, long long st_, int bits, int G,
                            unsigned char *codes, void *scales, void *zeros,
                            long long osb, long long osh, unsigned *status, const int *exact_blocks, int meta16, cudaStream_t st)
{
    KeyParams p;
    p.Wimg = Wimg; p.k = k; p.sb = sb; p.sh = sh; p.st = st_;
    p.codes = codes; p.scales = scales; p.zeros = zeros; p.osb = osb; p.osh = osh;
    p.B = batch; p.H = H; p.T = T; p.groups_per_bh = T / G;
    p.status = status;
    p.exact_blocks = exact_blocks;
#ifdef SQUAT_CHECKED
    {
        const unsigned long long es = dtype == SQUAT_BF16 ? 2 : 4, ms = meta16 ? 2 : 4;
        const long long ng = T / G;
        p.x_k = {k, (unsigned long long)((batch - 1) * sb + (H - 1) * sh + (long long)(T - 1) * st_ + D) * es};
        p.x_codes = {codes, (unsigned long long)((batch - 1) * osb + (H - 1) * osh + T) * (D * bits / 8)};
        const unsigned long long meta_elems = (unsigned long long)(((batch - 1) * osb + (H - 1) * osh) / G + ng) * D;
        p.x_scales = {scales, meta_elems * ms};
        p.x_zeros = {zeros, meta_elems * ms};
        p.x_img = {Wimg, (unsigned long long)H * TC_IMG_FLOATS * 4};
    }
#endif
    if ((long long)H * batch * (T / G) == 0) return SQUAT_OK;
    if (bits == 2) {
        if (G == 32) return launch_keys<2, 1>(p, dtype, meta16, st);
        if (G == 64) return launch_keys<2, 2>(p, dtype, meta16, st);
        if (G == 128) return launch_keys<2, 4>(p, dtype, meta16, st);
    } else if (bits == 4) {
        if (G == 32) return launch_keys<4, 1>(p, dtype, meta16, st);
        if (G == 64) return launch_keys<4, 2>(p, dtype, meta16, st);
        if (G == 128) return launch_keys<4, 4>(p, dtype, meta16, st);
    }
    return SQUAT_ERR_UNSUPPORTED;
}
