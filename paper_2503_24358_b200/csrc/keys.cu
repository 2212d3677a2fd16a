// Key quantization with error feedback: Algorithm 1, function Quant, with the update of
// Eq. (3) / Eq. (update_block) applied through the assembled matrix W (W[j'][j] multiplies the
// rounding error of channel j into channel j' > j), and the quantizer of Section 2.
//
// Mapping.  A group is G consecutive tokens of one (batch, head); its channels must be visited in
// order, and each channel's grid needs min/max over the group's tokens.  So: lane = token, one warp
// (G = 32) or a team of G/32 warps per group.  The 128 channels are processed in 4 blocks of 32:
//
//   left-looking trailing update (runtime loop, tiny code):
//       x_blk[tok][c] = k[tok][c] + sum_{j < block start} e_j[tok] * W[c][j]
//     a (32 tokens x J) x (J x 32 channels) product, register-tiled: each lane owns 8 tokens x 4
//     channels, reads 8 errors (two LDS.128 of the [channel][token] error store) and 4 entries of
//     W^T (one LDS.128) per j and issues 16 packed fma.rn.f32x2 -- 3 shared-memory reads per j
//     instead of 17 with one token per lane, which would make shared memory the bound.  The tile
//     is then transposed through shared memory to one token per lane for the sequential part.
//   in-block triangle (32 channels, unrolled so every register index is static; the same code
//   serves all 4 blocks):
//       m, M  = warp min / max (redux.sync on f32)         -> scale = (M-m)/L, zero = m
//       c     = rint((x_j - m)/scale), decided exactly through the remainder c*scale - (x_j - m)
//       e     = fma(c, scale, -(x_j - m))                   (= deq(qtz(x_j)) - x_j)
//       x_j' += e * W[j'][j]  for the later channels j' of the block; e goes to shared memory.
//
// The update matrix of the CTA's current head is kept in shared memory as 4 column panels
// (panel b = W^T[0 .. 32b+31][32b .. 32b+31], 40 KB in all: only the lower triangle is ever read).
// CTAs are persistent: each takes a contiguous range of groups ordered head-major, so W is
// reloaded only when the range crosses a head.  14 warps per SM x 2 rounds cover the 27.7 groups
// per SM of the 32-head x 4096-token workload.
//
// Work per key vector: 8128 fp32 FMA (dense triangle, g = 1) -> bound by the FP32 pipes, not HBM.
#include "squat_internal.cuh"

namespace {

constexpr int D = SQUAT_D;
constexpr int BLK = 32;                   // channels per block
constexpr int NBLK = D / BLK;             // 4
constexpr int PANEL_FLOATS = BLK * BLK * (NBLK * (NBLK + 1) / 2);   // 10 blocks of 32 x 32
constexpr int E_ROWS = D - BLK;           // errors of the last block are never read
constexpr float kMagic = 12582912.0f;     // 1.5 * 2^23
constexpr int KEY_WARPS = 14;
constexpr int KEY_THREADS = KEY_WARPS * 32;

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

struct KeyParams {
    const float *Wt;          // [H, D, D] transposed update matrices: Wt[j][j'] = W[j'][j]
    const void *k;
    long long sb, sh, st;     // element strides of k
    unsigned char *codes;
    float *scales, *zeros;
    long long osb, osh;       // output strides in tokens
    int B, H, T;
    int groups_per_bh;        // T / G
    long long total_groups;   // H * B * groups_per_bh, ordered (h, b, grp)
    unsigned *status;
    int exact_blocks;         // leading 32-channel blocks that no earlier channel corrects (see sweep_block)
};

// One lane's share of a 32-token x 32-channel block in the trailing-update layout: 8 tokens x 4 channels
// (tokens 8 tr .. 8 tr + 7, channels 4 cr .. 4 cr + 3 with tr = lane >> 3, cr = lane & 7).  The shape is chosen
// for the shared-memory pipe: 8 consecutive lanes share their token rows, so the two 16-byte reads of the
// error rows cost 2.5 cycles each instead of 4, and only the one read of W^T has 8 different addresses.
template <bool BF16>
struct RawTile {
    uint2 v[BF16 ? 8 : 16];     // per token: 4 channels = 8 B (bf16) or 16 B (f32)
};

template <bool BF16>
__device__ __forceinline__ void load_tile(RawTile<BF16> &r, const void *row0, long long st, int chan)
{
    // row0: first of the lane's 8 consecutive tokens; st: token stride in elements; chan: first channel
    if (BF16) {
        const __nv_bfloat16 *p = reinterpret_cast<const __nv_bfloat16 *>(row0) + chan;
#pragma unroll
        for (int i = 0; i < 8; ++i) r.v[i] = __ldg(reinterpret_cast<const uint2 *>(p + i * st));
    } else {
        const float *p = reinterpret_cast<const float *>(row0) + chan;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint4 t = ldg128(p + i * st);
            r.v[2 * i] = make_uint2(t.x, t.y);
            r.v[2 * i + 1] = make_uint2(t.z, t.w);
        }
    }
}

template <bool BF16>
__device__ __forceinline__ void unpack_tile(const RawTile<BF16> &r, u64 (&acc)[8][2])
{
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        if (BF16) {
            acc[i][0] = pack2(bf16lo_to_f32(r.v[i].x), bf16hi_to_f32(r.v[i].x));
            acc[i][1] = pack2(bf16lo_to_f32(r.v[i].y), bf16hi_to_f32(r.v[i].y));
        } else {
            acc[i][0] = pack2(__uint_as_float(r.v[2 * i].x), __uint_as_float(r.v[2 * i].y));
            acc[i][1] = pack2(__uint_as_float(r.v[2 * i + 1].x), __uint_as_float(r.v[2 * i + 1].y));
        }
    }
}

// The sequential part: the 32 channels of one block, one token per lane, values in xp (16 packed pairs).
// For every channel: grid from the warp (team) min / max, rounding decision, error e; e is pushed onto the
// later channels of the block through the diagonal 32 x 32 block of W^T and stored for the later blocks.
//
// Rounding decision.  t = (x - m) / scale is formed as (x - m) * L * rcp(M - m) with the hardware reciprocal,
// so c0 = rint(t) can be off by one when t is within ~1e-6 of a rounding midpoint.  Channels that earlier
// channels have corrected hold generic float32 values and such near-ties are as rare as that bound; but
// channels nothing has corrected yet (the first g channels, or all of them when W = 0) hold raw bf16 / f32
// inputs, where exact ties are structural (x exactly half way between min and max).  For those blocks
// (EXACT) the remainder e0 = c0*scale - (x - m), which is exact next to a midpoint, is compared with
// +-scale/2: that settles the rounding exactly as real arithmetic on the stored float32 scale would, ties
// going to the even code (the threshold of an odd c0 is one ulp lower, so "remainder == scale/2" moves it).
template <int BITS, int NW, bool EXACT>
__device__ __forceinline__ void sweep_block(u64 (&xp)[BLK / 2], const float *diag, float *Eblk, bool store_e,
                                            int lane, int team, int wteam, float2 *red, float2 *park,
                                            uint32_t (&cw)[BLK * BITS / 32], float &my_scale, float &my_zero)
{
    constexpr float L = float((1 << BITS) - 1);
    constexpr int PER_ACC = 16 / BITS;              // codes accumulated exactly in one float (16 bits of mantissa)
    float cacc[BLK / PER_ACC];
#pragma unroll
    for (int jj = 0; jj < BLK; ++jj) {
        const float xj = (jj & 1) ? hi_of(xp[jj >> 1]) : lo_of(xp[jj >> 1]);
        float m = warp_min(xj);
        float Mx = warp_max(xj);
        if (NW > 1) {
            float2 *slot = red + (team * 2 + (jj & 1)) * NW;
            if (lane == 0) slot[wteam] = make_float2(m, Mx);
            team_barrier(1 + team, 32 * NW);
#pragma unroll
            for (int w = 0; w < NW; ++w) {
                const float2 o = slot[w];
                m = fminf(m, o.x);
                Mx = fmaxf(Mx, o.y);
            }
        }
        const float rng = __fsub_rn(Mx, m);
        const float dlt = __fsub_rn(xj, m);
        const float dltL = __fmul_rn(dlt, L);
        float rcp;
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(rcp) : "f"(fmaxf(rng, 1e-30f)));   // constant group: dlt = 0 -> code 0
        const float scale = div_by_levels<BITS>(rng);
        const float y0 = __fmaf_rn(dltL, rcp, kMagic);
        float c = __fsub_rn(y0, kMagic);
        float e = __fmaf_rn(c, scale, -dlt);
        if (EXACT) {
            const float thr = __uint_as_float(__float_as_uint(0.5f * scale) - (__float_as_uint(y0) & 1u));
            const float adj = (e > thr) ? -1.0f : ((e < -thr) ? 1.0f : 0.0f);
            c = __fadd_rn(c, adj);
            e = __fmaf_rn(adj, scale, e);
        }
        // pack the code arithmetically: sum of c * 2^(BITS k) is exact in float32 up to 16 bits
        if (jj % PER_ACC == 0) cacc[jj / PER_ACC] = c;
        else cacc[jj / PER_ACC] = __fmaf_rn(c, float(1 << ((jj % PER_ACC) * BITS)), cacc[jj / PER_ACC]);
        park[jj] = make_float2(scale, m);               // same value from every lane; lane jj picks it up below
        if (store_e) Eblk[jj * 32] = e;
        const u64 ee = pack2(e, e);
        const float *wrow = diag + jj * BLK;
#pragma unroll
        for (int q = (jj + 1) / 4; q < BLK / 4; ++q) {
            const ulonglong2 wv = *reinterpret_cast<const ulonglong2 *>(wrow + 4 * q);
            if (2 * q >= (jj + 1) / 2) xp[2 * q] = ffma2(ee, wv.x, xp[2 * q]);
            xp[2 * q + 1] = ffma2(ee, wv.y, xp[2 * q + 1]);
        }
    }
    __syncwarp();
    const float2 sz = park[lane];
    my_scale = sz.x;
    my_zero = sz.y;
    __syncwarp();
#pragma unroll
    for (int w = 0; w < BLK * BITS / 32; ++w)
        cw[w] = (uint32_t)__float2int_rn(cacc[2 * w]) | ((uint32_t)__float2int_rn(cacc[2 * w + 1]) << 16);
}

template <int BITS, int NW, bool BF16>
__global__ void __launch_bounds__(KEY_THREADS, 1) quant_keys_kernel(const KeyParams p)
{
    constexpr int G = 32 * NW;
    constexpr int NTEAMS = KEY_WARPS / NW;
    constexpr int WORDS_PER_BLK = BLK * BITS / 32;       // 2 (2-bit) or 4 (4-bit)
    extern __shared__ __align__(16) float smem[];
    float *Wp = smem;                                    // 4 column panels, PANEL_FLOATS
    float *Eall = smem + PANEL_FLOATS;                   // [KEY_WARPS][E_ROWS][32]
    float2 *red = reinterpret_cast<float2 *>(Eall + KEY_WARPS * E_ROWS * 32);   // [NTEAMS][2][NW]
    float2 *park = red + NTEAMS * 2 * NW + (threadIdx.x >> 5) * BLK;             // [KEY_WARPS][BLK] (scale, zero) of a block

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int team = warp / NW;
    const int wteam = warp % NW;
    float *Ew = Eall + warp * (E_ROWS * 32) + lane;      // this lane's column of the warp's error store

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
            // panel cb holds rows j = 0 .. 32 cb + 31 of W^T restricted to columns 32 cb .. 32 cb + 31
            const float *src = p.Wt + (long long)h * D * D;
            for (int i = threadIdx.x; i < PANEL_FLOATS / 4; i += KEY_THREADS) {
                int f = i * 4, cb = 0;
                while (f >= BLK * BLK * (cb + 1)) { f -= BLK * BLK * (cb + 1); ++cb; }
                const int j = f / BLK, c = f % BLK;
                reinterpret_cast<float4 *>(Wp)[i] = __ldg(reinterpret_cast<const float4 *>(src + j * D + cb * BLK + c));
            }
        }
        __syncthreads();

        if (team < NTEAMS) {
            for (long long gi = pos + team; gi < seg_end; gi += NTEAMS) {
                const long long in_head = gi - (long long)h * groups_per_head;
                const int b = (int)(in_head / p.groups_per_bh);
                const int grp = (int)(in_head % p.groups_per_bh);
                const int tok = grp * G + wteam * 32 + lane;
                const long long out_tok0 = (long long)b * p.osb + (long long)h * p.osh;
                float *sc_out = p.scales + (out_tok0 / G + grp) * D;
                float *zr_out = p.zeros + (out_tok0 / G + grp) * D;
                unsigned char *cp = p.codes + (out_tok0 + tok) * (D * BITS / 8);

                // trailing-update layout: this lane owns tokens 8 tr .. 8 tr + 7 and channels 4 cr .. 4 cr + 3 of a block
                const int tr = lane >> 3, cr = lane & 7;
                const long long row0_off = (long long)b * p.sb + (long long)h * p.sh +
                                           (long long)(grp * G + wteam * 32 + 8 * tr) * p.st;
                const void *row0 = BF16 ? static_cast<const void *>(reinterpret_cast<const __nv_bfloat16 *>(p.k) + row0_off)
                                        : static_cast<const void *>(reinterpret_cast<const float *>(p.k) + row0_off);
                RawTile<BF16> raw;
                load_tile<BF16>(raw, row0, p.st, 4 * cr);

                for (int blk = 0; blk < NBLK; ++blk) {
                    const float *panel = Wp + (blk * (blk + 1) / 2) * (BLK * BLK);
                    const int nprev = blk * BLK;
                    u64 xp[BLK / 2];
                    {
                        // ---- left-looking update from all earlier channels, as a register-tiled product:
                        //      acc[token][channel pair] = k + sum_j e_j[token] * W^T[j][channel]
                        u64 acc[8][2];
                        unpack_tile<BF16>(raw, acc);
                        if (blk + 1 < NBLK) load_tile<BF16>(raw, row0, p.st, (blk + 1) * BLK + 4 * cr);   // prefetch
                        const float *e_ptr = Ew - lane + 8 * tr;          // E[j][8 tr .. 8 tr + 7]
                        const float *w_ptr = panel + 4 * cr;              // W^T[j][4 cr .. 4 cr + 3]
                        // software-pipelined over j: the operands of the next 2 steps are loaded while the current 2
                        // steps' 32 packed FMAs issue (warps issue in order, so the loads must be hoisted by hand)
                        constexpr int PF = 2;
                        float4 ea[PF][2], eb[PF][2];
                        ulonglong2 wa[PF], wb[PF];
                        auto loadn = [&](float4 (&ev)[PF][2], ulonglong2 (&wv)[PF], int j0) {
#pragma unroll
                            for (int u = 0; u < PF; ++u) {
                                ev[u][0] = *reinterpret_cast<const float4 *>(e_ptr + (j0 + u) * 32);
                                ev[u][1] = *reinterpret_cast<const float4 *>(e_ptr + (j0 + u) * 32 + 4);
                                wv[u] = *reinterpret_cast<const ulonglong2 *>(w_ptr + (j0 + u) * BLK);
                            }
                        };
                        auto fman = [&](const float4 (&ev)[PF][2], const ulonglong2 (&wv)[PF]) {
#pragma unroll
                            for (int u = 0; u < PF; ++u) {
                                const float e[8] = {ev[u][0].x, ev[u][0].y, ev[u][0].z, ev[u][0].w,
                                                    ev[u][1].x, ev[u][1].y, ev[u][1].z, ev[u][1].w};
#pragma unroll
                                for (int i = 0; i < 8; ++i) {
                                    const u64 ee = pack2(e[i], e[i]);
                                    acc[i][0] = ffma2(ee, wv[u].x, acc[i][0]);
                                    acc[i][1] = ffma2(ee, wv[u].y, acc[i][1]);
                                }
                            }
                        };
                        if (nprev > 0) {
                            loadn(ea, wa, 0);
#pragma unroll 1
                            for (int j = 0; j < nprev; j += 2 * PF) {        // nprev is a multiple of 32
                                loadn(eb, wb, j + PF);
                                fman(ea, wa);
                                loadn(ea, wa, (j + 2 * PF < nprev) ? j + 2 * PF : j);   // last reload: redundant, in range
                                fman(eb, wb);
                            }
                        }
                        // ---- transpose to one token per lane through a 4 KB staging tile (the error rows this
                        //      block is about to fill; for the last block, rows 0..31, which nothing reads any more).
                        //      16-byte chunks are swizzled with the token index: 8 consecutive lanes write one token's
                        //      8 chunks (one 128-byte row), 8 consecutive tokens read 8 different chunks.
                        float *stage = Ew - lane + ((blk + 1 < NBLK) ? nprev * 32 : 0);
                        __syncwarp();
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const int tok = 8 * tr + i;
                            *reinterpret_cast<ulonglong2 *>(stage + tok * 32 + 4 * (cr ^ i)) = make_ulonglong2(acc[i][0], acc[i][1]);
                        }
                        __syncwarp();
#pragma unroll
                        for (int q = 0; q < BLK / 4; ++q) {
                            const ulonglong2 v = *reinterpret_cast<const ulonglong2 *>(stage + lane * 32 + 4 * (q ^ (lane & 7)));
                            xp[2 * q] = v.x;
                            xp[2 * q + 1] = v.y;
                        }
                        __syncwarp();
                    }

                    // ---- sequential sweep over the block's 32 channels ------------------------
                    const float *diag = panel + nprev * BLK;
                    float *Eblk = Ew + nprev * 32;
                    uint32_t cw[WORDS_PER_BLK];
                    float my_scale = 0.0f, my_zero = 0.0f;
                    if (blk < p.exact_blocks)
                        sweep_block<BITS, NW, true>(xp, diag, Eblk, blk + 1 < NBLK, lane, team, wteam, red, park, cw, my_scale, my_zero);
                    else
                        sweep_block<BITS, NW, false>(xp, diag, Eblk, blk + 1 < NBLK, lane, team, wteam, red, park, cw, my_scale, my_zero);

                    // ---- this block's outputs -----------------------------------------------
                    if (WORDS_PER_BLK == 2)
                        *reinterpret_cast<uint2 *>(cp + blk * (BLK * BITS / 8)) = make_uint2(cw[0], cw[1]);
                    else
                        *reinterpret_cast<uint4 *>(cp + blk * (BLK * BITS / 8)) =
                            make_uint4(cw[0], cw[1], cw[WORDS_PER_BLK > 2 ? 2 : 0], cw[WORDS_PER_BLK > 2 ? 3 : 0]);
                    if (wteam == 0) {
                        sc_out[blk * BLK + lane] = my_scale;
                        zr_out[blk * BLK + lane] = my_zero;
                        if (!(my_scale > 0.0f && my_scale < __int_as_float(0x7f800000)))
                            atomicOr(p.status, my_scale == 0.0f ? SQUAT_FLAG_ZERO_RANGE : SQUAT_FLAG_NONFINITE);
                    }
                }
            }
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
    constexpr int NTEAMS = KEY_WARPS / NW;
    const size_t smem = sizeof(float) * (PANEL_FLOATS + KEY_WARPS * E_ROWS * 32) + sizeof(float2) * (NTEAMS * 2 * NW + KEY_WARPS * BLK);
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
                            long long osb, long long osh, unsigned *status, int exact_blocks, cudaStream_t st)
{
    KeyParams p;
    p.Wt = Wt; p.k = k; p.sb = sb; p.sh = sh; p.st = st_;
    p.codes = codes; p.scales = scales; p.zeros = zeros; p.osb = osb; p.osh = osh;
    p.B = batch; p.H = H; p.T = T; p.groups_per_bh = T / G;
    p.total_groups = (long long)H * batch * (T / G);
    p.status = status;
    p.exact_blocks = exact_blocks;
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
