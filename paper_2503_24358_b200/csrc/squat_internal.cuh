// Internal declarations shared by the translation units of libsquat (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "../../include/squat.h"

#define SQUAT_D 128   // the only head dimension the key path and the subspace build are built for
#define SQUAT_LOWRANK_MAX_R 8   // largest subspace rank the rank-r form of the key quantizer is built for (keys_lowrank.cu)

struct squat_subspace {
    int n_kv_heads;
    int head_dim;
    int device;
    int gram_chunks_cap;   // capacity (in row chunks per head) of gram_partial
    int *exact_blocks;     // device word: leading 32-channel blocks of W that receive no correction (4 when W = 0); written in
                           // stream order by the kernel that packs W, read by the key kernel, so it always belongs to the W it is
                           // launched with (a host-side copy could be overtaken by a build enqueued from another thread or stream)
    float *Wt;             // [H, d, d] float32, Wt[h][j][j'] = W[j'][j]  (row j = update vector of channel j)
    float *Wimg;           // [H, d * d] the same matrices as the key kernel stages them in shared memory (see keys.cu)
    float *lr_table;       // [H, d, 2 * SQUAT_LOWRANK_MAX_R] rows [v_j | c_j] of the rank-r form of W (keys_lowrank.cu)
    int lowrank_r;         // > 0: lr_table describes the same update as Wt (set by the SVD builds with g = 1 and a small rank);
                           // host-side, read when a key call is enqueued: calls on one handle are issued in execution order
    int prefer_dense;      // 1: squat_quantize_keys uses the dense kernel even when lr_table is valid
    double *gram;          // [H, d, d] Gram matrices
    double *gram_partial;  // [chunks, H, d, d] per-chunk partial Gram matrices (deterministic reduction)
    double *eigval;        // [H, d] descending
    double *eigvec;        // [H, d, d], row i = eigenvector i
    int *eig_sweeps;       // [H] sweeps of the last eigen-decomposition
    unsigned *status;      // device status word of this device
    // host path only (created on its first call): two side streams and the events that order them
    cudaStream_t side[2];
    cudaEvent_t ev[8];     // q up, k up, keys done, key outputs down, v chunks up (4)
    bool side_ready;
};

// ---- host-side helpers (api.cu) ------------------------------------------------------
int squat_cuda_fail(cudaError_t e);          // records the error text, returns SQUAT_ERR_CUDA
unsigned *squat_status_word();               // device address of the status word of the current device
void squat_count_launch(unsigned n = 1);
#define SQUAT_CUDA(call) do { cudaError_t e__ = (call); if (e__ != cudaSuccess) return squat_cuda_fail(e__); } while (0)
#define SQUAT_LAUNCH_CHECK() do { cudaError_t e__ = cudaGetLastError(); if (e__ != cudaSuccess) return squat_cuda_fail(e__); } while (0)

// ---- kernel launchers (one per .cu) ---------------------------------------------------
int squat_launch_gram(squat_subspace *s, const void *q, int dtype, int n_q_heads, int n_tokens,
                      long long stride_h, long long stride_t, cudaStream_t st);
int squat_launch_eig(squat_subspace *s, cudaStream_t st);
int squat_launch_assemble(squat_subspace *s, int rank_r, double lambda, int block_g, int left_rows, int exact_blocks, cudaStream_t st);
int squat_launch_power(squat_subspace *s, const double *start, long long start_stride_h, int rank_r, int iters,
                       double lambda, cudaStream_t st);

int squat_launch_lowrank_tables(squat_subspace *s, int rank_r, double lambda, cudaStream_t st);
int squat_launch_quant_keys_lowrank(const float *table, const void *k, int dtype, int batch, int H, int T,
                                    long long sb, long long sh, long long st_, int bits, int G,
                                    unsigned char *codes, void *scales, void *zeros,
                                    long long osb, long long osh, unsigned *status, int meta16, cudaStream_t st);
int squat_launch_pack_update_matrices(const float *Wt, float *Wimg, int H, int exact_blocks, int *exact_blocks_dev, cudaStream_t st);
int squat_launch_quant_keys(const float *Wimg, const void *k, int dtype, int batch, int H, int T,
                            long long sb, long long sh, long long st_, int bits, int G,
                            unsigned char *codes, void *scales, void *zeros,
                            long long osb, long long osh, unsigned *status, const int *exact_blocks_dev, int meta16, cudaStream_t st);
int squat_launch_quant_values(const void *v, int dtype, int batch, int H, int T, int d,
                              long long sb, long long sh, long long st_, int bits, int G,
                              unsigned char *codes, void *scales, void *zeros,
                              long long osb, long long osh, unsigned *status, int meta16, cudaStream_t st);
size_t squat_attention_workspace_floats(int batch, int n_q_heads, int n_tokens);
int squat_launch_decode_attention(const void *q, int q_dtype, int batch, int Hq, int H, int T,
                                  const unsigned char *kc, const void *ks, const void *kz,
                                  const unsigned char *vc, const void *vs, const void *vz,
                                  long long csb, long long csh, int bits, int G,
                                  const void *k_res, const void *v_res, int res_dtype, int R,
                                  float scale, float *out, float *workspace,
                                  const float *rope_table, int rope_blocks, long long first_pos, int meta16, cudaStream_t st);
int squat_launch_dequant(int kind, const unsigned char *codes, const void *scales, const void *zeros,
                         int batch, int H, int T, int d, int bits, int G, long long isb, long long ish,
                         void *out, int out_dtype, int meta16, cudaStream_t st);

// ---- the bounds-checked build ----------------------------------------------------------
// Compiled with -DSQUAT_CHECKED (build.py --checked -> libsquat_checked.so) the key and value kernels test every
// global, shared-memory and tensor-memory address they form (and the shared-memory windows of the matrix descriptors
// they hand to the tensor core) against the extent of the buffer or region it belongs to; an address outside sets
// SQUAT_FLAG_BOUNDS in the device status word and the access is skipped -- never a trap.  The stand-in for a memory
// checker on machines where none can be run; the tests drive small and ragged cases through it.  In the normal build
// every macro below folds to `true` and the extents do not exist.
#ifdef SQUAT_CHECKED
struct SqExtent {
    const void *base;
    unsigned long long bytes;
};
__device__ __forceinline__ bool sq_chk(bool ok, unsigned *status)
{
    if (!ok) atomicOr(status, SQUAT_FLAG_BOUNDS);
    return ok;
}
__device__ __forceinline__ bool sq_inside(const void *ptr, unsigned long long n, const void *base, unsigned long long bytes)
{
    const unsigned long long a = (unsigned long long)ptr, b = (unsigned long long)base;
    return a >= b && a + n <= b + bytes;
}
#define SQ_CHK_G(status, ptr, n, ext) sq_chk(sq_inside((ptr), (n), (ext).base, (ext).bytes), (status))       /* global memory */
#define SQ_CHK_R(status, ptr, n, base, bytes) sq_chk(sq_inside((ptr), (n), (base), (bytes)), (status))      /* a region (shared memory) */
#define SQ_CHK_C(status, cond) sq_chk((cond), (status))                                                      /* any condition */
#else
#define SQ_CHK_G(status, ptr, n, ext) true
#define SQ_CHK_R(status, ptr, n, base, bytes) true
#define SQ_CHK_C(status, cond) true
#endif

// ---- small device helpers --------------------------------------------------------------
__device__ __forceinline__ float bf16lo_to_f32(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

__device__ __forceinline__ uint4 ldg128(const void *p) { return __ldg(reinterpret_cast<const uint4 *>(p)); }
