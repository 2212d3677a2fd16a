// extern "C" entry points of libsquat: argument validation, handle management and the
// stream-ordered launch sequences.  All arithmetic of the method lives in the kernels.
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "squat_internal.cuh"

namespace {

constexpr int D = SQUAT_D;
constexpr int MAX_DEVICES = 64;

thread_local char g_cuda_error[256] = "";
std::atomic<unsigned long long> g_launches{0};

__device__ unsigned g_status_word = 0;
unsigned *g_status_ptr[MAX_DEVICES] = {nullptr};

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
// A handle's memory lives on the device that was current when it was created; its calls must run there.
bool on_handle_device(const squat_subspace *s)
{
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == s->device;
}
bool valid_dtype(int dt) { return dt == SQUAT_F32 || dt == SQUAT_BF16; }
size_t elem_size(int dt) { return dt == SQUAT_BF16 ? 2 : 4; }

// Shared checks of the two quantizers.  Strides are in elements (input) / tokens (output).
int check_quant_args(const void *x, int dtype, int batch, int H, int T, int d, long long sb, long long sh,
                     long long st, int bits, int G, const void *codes, const void *scales, const void *zeros,
                     long long osb, long long osh)
{
    if (!valid_dtype(dtype) || batch < 0 || H <= 0 || T < 0 || d <= 0) return SQUAT_ERR_INVALID_ARG;
    const bool empty = batch == 0 || T == 0;             // nothing will be read or written
    if (!empty && (!x || !codes || !scales || !zeros)) return SQUAT_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(codes) || !aligned16(scales) || !aligned16(zeros)) return SQUAT_ERR_INVALID_ARG;
    if (bits != 2 && bits != 4) return SQUAT_ERR_UNSUPPORTED;
    if (G != 32 && G != 64 && G != 128) return SQUAT_ERR_UNSUPPORTED;
    if (sb < 0 || sh < 0 || st < d || osb < 0 || osh < 0) return SQUAT_ERR_INVALID_ARG;
    const long long vec = 16 / (long long)elem_size(dtype);       // 128-bit loads
    if (sb % vec || sh % vec || st % vec) return SQUAT_ERR_INVALID_ARG;
    return SQUAT_OK;
}

// The rank-r form of the update (keys_lowrank.cu) exists for element-wise updates with a small rank: its tables are
// made from the eigen-pairs right after the eigensolver.  Every other build leaves the handle on the dense kernel.
int lowrank_tables_if_small(squat_subspace *s, int rank_r, double lambda, int block_g, cudaStream_t st)
{
    s->lowrank_r = 0;
    if (block_g != 1 || rank_r < 1 || rank_r > SQUAT_LOWRANK_MAX_R || !(lambda > 0.0)) return SQUAT_OK;
    const int rc = squat_launch_lowrank_tables(s, rank_r, lambda, st);
    if (rc == SQUAT_OK) s->lowrank_r = rank_r;
    return rc;
}

}  // namespace

int squat_cuda_fail(cudaError_t e)
{
    snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
    return SQUAT_ERR_CUDA;
}

void squat_count_launch(unsigned n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

unsigned *squat_status_word()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return nullptr;
    if (!g_status_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) return nullptr;
        g_status_ptr[dev] = static_cast<unsigned *>(p);
    }
    return g_status_ptr[dev];
}

extern "C" {

const char *squat_status_string(int status)
{
    switch (status) {
        case SQUAT_OK: return "ok";
        case SQUAT_ERR_INVALID_ARG: return "invalid argument";
        case SQUAT_ERR_SHAPE: return "shape does not divide as required";
        case SQUAT_ERR_UNSUPPORTED: return "configuration not built";
        case SQUAT_ERR_ALLOC: return "device allocation failed";
        case SQUAT_ERR_CUDA: return "CUDA runtime error";
        case SQUAT_ERR_NUMERIC: return "numerical failure";
        default: return "unknown status";
    }
}

const char *squat_last_cuda_error(void) { return g_cuda_error; }

unsigned long long squat_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int squat_subspace_create(int n_kv_heads, int head_dim, squat_subspace **out)
{
    if (!out) return SQUAT_ERR_INVALID_ARG;
    *out = nullptr;
    if (n_kv_heads <= 0 || n_kv_heads > 65535 || head_dim <= 0) return SQUAT_ERR_INVALID_ARG;
    if (head_dim != D) return SQUAT_ERR_UNSUPPORTED;
    squat_subspace *s = new (std::nothrow) squat_subspace();
    if (!s) return SQUAT_ERR_ALLOC;
    memset(s, 0, sizeof(*s));
    s->n_kv_heads = n_kv_heads;
    s->head_dim = head_dim;
    int sms = 148;
    if (cudaGetDevice(&s->device) != cudaSuccess) { delete s; return SQUAT_ERR_CUDA; }
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, s->device);
    s->gram_chunks_cap = (2 * sms) / n_kv_heads;        // 2 resident CTAs per SM: one wave
    if (s->gram_chunks_cap < 1) s->gram_chunks_cap = 1;
    const size_t hdd = (size_t)n_kv_heads * D * D;
    // one allocation, carved up (256-byte aligned pieces)
    size_t off = 0;
    auto carve = [&](size_t bytes) { size_t o = off; off += (bytes + 255) / 256 * 256; return o; };
    const size_t o_wt = carve(hdd * sizeof(float));
    const size_t o_img = carve(hdd * sizeof(float));
    const size_t o_gram = carve(hdd * sizeof(double));
    const size_t o_part = carve(hdd * sizeof(double) * s->gram_chunks_cap);
    const size_t o_val = carve((size_t)n_kv_heads * D * sizeof(double));
    const size_t o_vec = carve(hdd * sizeof(double));
    const size_t o_swp = carve((size_t)n_kv_heads * sizeof(int));
    const size_t o_exact = carve(sizeof(int));
    const size_t o_lr = carve((size_t)n_kv_heads * D * 2 * SQUAT_LOWRANK_MAX_R * sizeof(float));
    char *base = nullptr;
    if (cudaMalloc(&base, off) != cudaSuccess) { cudaGetLastError(); delete s; return SQUAT_ERR_ALLOC; }
    if (cudaMemset(base, 0, off) != cudaSuccess) { cudaFree(base); delete s; return SQUAT_ERR_CUDA; }
    s->Wt = reinterpret_cast<float *>(base + o_wt);
    s->Wimg = reinterpret_cast<float *>(base + o_img);
    s->gram = reinterpret_cast<double *>(base + o_gram);
    s->gram_partial = reinterpret_cast<double *>(base + o_part);
    s->eigval = reinterpret_cast<double *>(base + o_val);
    s->eigvec = reinterpret_cast<double *>(base + o_vec);
    s->eig_sweeps = reinterpret_cast<int *>(base + o_swp);
    s->exact_blocks = reinterpret_cast<int *>(base + o_exact);
    s->lr_table = reinterpret_cast<float *>(base + o_lr);
    const int all_exact = D / 32;        // W starts as zero: every channel is uncorrected
    if (cudaMemcpy(s->exact_blocks, &all_exact, sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess) { cudaFree(base); delete s; return SQUAT_ERR_CUDA; }
    s->status = squat_status_word();
    if (!s->status) { cudaFree(base); delete s; return SQUAT_ERR_CUDA; }
    *out = s;
    return SQUAT_OK;
}

int squat_subspace_destroy(squat_subspace *s)
{
    if (!s) return SQUAT_OK;
    if (s->side_ready) {
        for (int i = 0; i < 2; ++i) cudaStreamDestroy(s->side[i]);
        for (int i = 0; i < 8; ++i) cudaEventDestroy(s->ev[i]);
    }
    cudaError_t e = cudaFree(s->Wt);     // Wt is the base of the single allocation
    delete s;
    return e == cudaSuccess ? SQUAT_OK : squat_cuda_fail(e);
}

int squat_build_subspace(squat_subspace *s, const void *q, int dtype, int n_q_heads, int n_tokens,
                         long long stride_h, long long stride_t, int rank_r, double lambda,
                         int block_g, void *stream)
{
    if (!s || !q || !valid_dtype(dtype) || !aligned16(q)) return SQUAT_ERR_INVALID_ARG;
    if (!on_handle_device(s)) return SQUAT_ERR_INVALID_ARG;     // the handle belongs to another device
    if (n_q_heads <= 0 || n_tokens <= 0) return SQUAT_ERR_INVALID_ARG;
    if (n_q_heads % s->n_kv_heads != 0) return SQUAT_ERR_SHAPE;
    if (rank_r < 0 || rank_r > D) return SQUAT_ERR_INVALID_ARG;
    if ((long long)rank_r > (long long)n_tokens * (n_q_heads / s->n_kv_heads)) return SQUAT_ERR_SHAPE;
    if (!(lambda >= 0.0) || !std::isfinite(lambda)) return SQUAT_ERR_INVALID_ARG;
    if (block_g <= 0 || D % block_g != 0) return SQUAT_ERR_SHAPE;
    const long long vec = 16 / (long long)elem_size(dtype);
    if (stride_t < D || stride_h < 0 || stride_t % vec || stride_h % vec) return SQUAT_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int rc = squat_launch_gram(s, q, dtype, n_q_heads, n_tokens, stride_h, stride_t, st);
    if (rc != SQUAT_OK) return rc;
    rc = squat_launch_eig(s, st);
    if (rc != SQUAT_OK) return rc;
    rc = lowrank_tables_if_small(s, rank_r, lambda, block_g, st);
    if (rc != SQUAT_OK) return rc;
    // channels of the first g-block are never corrected; with r = 0 or lambda = 0, W = 0 and none is
    const int exact = (rank_r == 0 || lambda == 0.0) ? D / 32 : (block_g + 31) / 32;
    return squat_launch_assemble(s, rank_r, lambda, block_g, 0, exact, st);
}

int squat_build_subspace_from_gram(squat_subspace *s, const double *gram, int rank_r, double lambda, int block_g,
                                   void *stream)
{
    if (!s || !gram || !aligned16(gram)) return SQUAT_ERR_INVALID_ARG;
    if (!on_handle_device(s)) return SQUAT_ERR_INVALID_ARG;     // the handle belongs to another device
    if (rank_r < 0 || rank_r > D) return SQUAT_ERR_INVALID_ARG;
    if (!(lambda >= 0.0) || !std::isfinite(lambda)) return SQUAT_ERR_INVALID_ARG;
    if (block_g <= 0 || D % block_g != 0) return SQUAT_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (gram != s->gram)
        SQUAT_CUDA(cudaMemcpyAsync(s->gram, gram, (size_t)s->n_kv_heads * D * D * sizeof(double), cudaMemcpyDeviceToDevice, st));
    int rc = squat_launch_eig(s, st);
    if (rc != SQUAT_OK) return rc;
    rc = lowrank_tables_if_small(s, rank_r, lambda, block_g, st);
    if (rc != SQUAT_OK) return rc;
    const int exact = (rank_r == 0 || lambda == 0.0) ? D / 32 : (block_g + 31) / 32;
    return squat_launch_assemble(s, rank_r, lambda, block_g, 0, exact, st);
}

int squat_build_subspace_power(squat_subspace *s, const void *q, int dtype, int n_q_heads, int n_tokens,
                               long long stride_h, long long stride_t, int rank_r, double lambda, int block_g,
                               const double *start_block, long long start_stride_h, int iters, void *stream)
{
    if (!s || !q || !valid_dtype(dtype) || !aligned16(q)) return SQUAT_ERR_INVALID_ARG;
    if (!on_handle_device(s)) return SQUAT_ERR_INVALID_ARG;     // the handle belongs to another device
    if (n_q_heads <= 0 || n_tokens <= 0) return SQUAT_ERR_INVALID_ARG;
    if (n_q_heads % s->n_kv_heads != 0) return SQUAT_ERR_SHAPE;
    if (rank_r < 0 || rank_r > D) return SQUAT_ERR_INVALID_ARG;
    if (rank_r > 64) return SQUAT_ERR_UNSUPPORTED;
    if ((long long)rank_r > (long long)n_tokens * (n_q_heads / s->n_kv_heads)) return SQUAT_ERR_SHAPE;
    if (!(lambda >= 0.0) || !std::isfinite(lambda)) return SQUAT_ERR_INVALID_ARG;
    if (block_g <= 0 || D % block_g != 0) return SQUAT_ERR_SHAPE;
    if (iters < 0 || iters > 64 || start_stride_h < 0) return SQUAT_ERR_INVALID_ARG;
    if (rank_r > 0 && (!start_block || ((uintptr_t)start_block & 7u))) return SQUAT_ERR_INVALID_ARG;
    if (start_stride_h != 0 && start_stride_h < (long long)D * rank_r) return SQUAT_ERR_INVALID_ARG;
    const long long vec = 16 / (long long)elem_size(dtype);
    if (stride_t < D || stride_h < 0 || stride_t % vec || stride_h % vec) return SQUAT_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int rc = squat_launch_gram(s, q, dtype, n_q_heads, n_tokens, stride_h, stride_t, st);
    if (rc != SQUAT_OK) return rc;
    const bool no_update = rank_r == 0 || lambda == 0.0;
    s->lowrank_r = 0;                      // the iterated basis is no eigenbasis: dense kernel
    const int exact = no_update ? D / 32 : (block_g + 31) / 32;
    if (no_update) return squat_launch_assemble(s, 0, lambda, block_g, 0, exact, st);      // W = 0: nothing to iterate
    rc = squat_launch_power(s, start_block, start_stride_h, rank_r, iters, lambda, st);
    if (rc != SQUAT_OK) return rc;
    return squat_launch_assemble(s, rank_r, lambda, block_g, 64, exact, st);
}

int squat_build_subspace_power_from_gram(squat_subspace *s, const double *gram, int rank_r, double lambda, int block_g,
                                         const double *start_block, long long start_stride_h, int iters, void *stream)
{
    if (!s || !gram || !aligned16(gram)) return SQUAT_ERR_INVALID_ARG;
    if (!on_handle_device(s)) return SQUAT_ERR_INVALID_ARG;     // the handle belongs to another device
    if (rank_r < 0 || rank_r > D) return SQUAT_ERR_INVALID_ARG;
    if (rank_r > 64) return SQUAT_ERR_UNSUPPORTED;
    if (!(lambda >= 0.0) || !std::isfinite(lambda)) return SQUAT_ERR_INVALID_ARG;
    if (block_g <= 0 || D % block_g != 0) return SQUAT_ERR_SHAPE;
    if (iters < 0 || iters > 64 || start_stride_h < 0) return SQUAT_ERR_INVALID_ARG;
    if (rank_r > 0 && (!start_block || ((uintptr_t)start_block & 7u))) return SQUAT_ERR_INVALID_ARG;
    if (start_stride_h != 0 && start_stride_h < (long long)D * rank_r) return SQUAT_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (gram != s->gram)
        SQUAT_CUDA(cudaMemcpyAsync(s->gram, gram, (size_t)s->n_kv_heads * D * D * sizeof(double), cudaMemcpyDeviceToDevice, st));
    const bool no_update = rank_r == 0 || lambda == 0.0;
    s->lowrank_r = 0;                      // the iterated basis is no eigenbasis: dense kernel
    const int exact = no_update ? D / 32 : (block_g + 31) / 32;
    if (no_update) return squat_launch_assemble(s, 0, lambda, block_g, 0, exact, st);
    int rc = squat_launch_power(s, start_block, start_stride_h, rank_r, iters, lambda, st);
    if (rc != SQUAT_OK) return rc;
    return squat_launch_assemble(s, rank_r, lambda, block_g, 64, exact, st);
}

int squat_subspace_export(const squat_subspace *s, void *stream, float *W_host, double *gram_host,
                          double *eigval_host, double *eigvec_host)
{
    if (!s) return SQUAT_ERR_INVALID_ARG;
    if (!on_handle_device(s)) return SQUAT_ERR_INVALID_ARG;     // the handle belongs to another device
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t hdd = (size_t)s->n_kv_heads * D * D;
    std::vector<float> wt;
    if (W_host) {
        wt.resize(hdd);
        SQUAT_CUDA(cudaMemcpyAsync(wt.data(), s->Wt, hdd * sizeof(float), cudaMemcpyDeviceToHost, st));
    }
    if (gram_host) SQUAT_CUDA(cudaMemcpyAsync(gram_host, s->gram, hdd * sizeof(double), cudaMemcpyDeviceToHost, st));
    if (eigval_host) SQUAT_CUDA(cudaMemcpyAsync(eigval_host, s->eigval, (size_t)s->n_kv_heads * D * sizeof(double), cudaMemcpyDeviceToHost, st));
    if (eigvec_host) SQUAT_CUDA(cudaMemcpyAsync(eigvec_host, s->eigvec, hdd * sizeof(double), cudaMemcpyDeviceToHost, st));
    SQUAT_CUDA(cudaStreamSynchronize(st));
    if (W_host)
        for (int h = 0; h < s->n_kv_heads; ++h)
            for (int j = 0; j < D; ++j)
                for (int jp = 0; jp < D; ++jp)
                    W_host[((size_t)h * D + jp) * D + j] = wt[((size_t)h * D + j) * D + jp];
    return SQUAT_OK;
}

int squat_subspace_select_key_kernel(squat_subspace *s, int prefer_dense, int *lowrank_rank)
{
    if (!s || (prefer_dense != 0 && prefer_dense != 1)) return SQUAT_ERR_INVALID_ARG;
    s->prefer_dense = prefer_dense;
    if (lowrank_rank) *lowrank_rank = s->lowrank_r;
    return SQUAT_OK;
}

int squat_subspace_eig_sweeps(const squat_subspace *s, void *stream, int *sweeps_host)
{
    if (!s || !sweeps_host) return SQUAT_ERR_INVALID_ARG;
    if (!on_handle_device(s)) return SQUAT_ERR_INVALID_ARG;     // the handle belongs to another device
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SQUAT_CUDA(cudaMemcpyAsync(sweeps_host, s->eig_sweeps, (size_t)s->n_kv_heads * sizeof(int), cudaMemcpyDeviceToHost, st));
    SQUAT_CUDA(cudaStreamSynchronize(st));
    return SQUAT_OK;
}

int squat_subspace_import(squat_subspace *s, const float *W_host, void *stream)
{
    if (!s || !W_host) return SQUAT_ERR_INVALID_ARG;
    if (!on_handle_device(s)) return SQUAT_ERR_INVALID_ARG;     // the handle belongs to another device
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t hdd = (size_t)s->n_kv_heads * D * D;
    std::vector<float> wt(hdd);
    for (int h = 0; h < s->n_kv_heads; ++h)
        for (int j = 0; j < D; ++j)
            for (int jp = 0; jp < D; ++jp)
                wt[((size_t)h * D + j) * D + jp] = W_host[((size_t)h * D + jp) * D + j];
    // channel j' is uncorrected if row j' of W is zero in every head (channel 0 always is); the blocks that
    // hold the leading run of uncorrected channels need the exact rounding decision
    int uncorrected = D;
    for (int h = 0; h < s->n_kv_heads; ++h)
        for (int jp = 0; jp < uncorrected; ++jp)
            for (int j = 0; j < D; ++j)
                if (W_host[((size_t)h * D + jp) * D + j] != 0.0f) { uncorrected = jp; break; }
    const int exact = (uncorrected + 31) / 32;
    s->lowrank_r = 0;                      // an imported W comes without its factors: dense kernel
    SQUAT_CUDA(cudaMemcpyAsync(s->Wt, wt.data(), hdd * sizeof(float), cudaMemcpyHostToDevice, st));
    int rc = squat_launch_pack_update_matrices(s->Wt, s->Wimg, s->n_kv_heads, exact, s->exact_blocks, st);
    if (rc != SQUAT_OK) return rc;
    SQUAT_CUDA(cudaStreamSynchronize(st));
    return SQUAT_OK;
}

namespace {
int quantize_keys_impl(const squat_subspace *s, const void *k, int dtype, int batch, int n_kv_heads,
                       int n_tokens, int head_dim, long long stride_b, long long stride_h,
                       long long stride_t, int bits, int group_size, unsigned char *codes,
                       void *scales, void *zeros, long long out_stride_b, long long out_stride_h, int meta16,
                       void *stream)
{
    if (!s) return SQUAT_ERR_INVALID_ARG;
    if (!on_handle_device(s)) return SQUAT_ERR_INVALID_ARG;     // the handle belongs to another device
    int rc = check_quant_args(k, dtype, batch, n_kv_heads, n_tokens, head_dim, stride_b, stride_h, stride_t, bits,
                              group_size, codes, scales, zeros, out_stride_b, out_stride_h);
    if (rc != SQUAT_OK) return rc;
    if (head_dim != D) return SQUAT_ERR_UNSUPPORTED;
    if (n_kv_heads != s->n_kv_heads) return SQUAT_ERR_SHAPE;
    if (n_tokens % group_size != 0 || out_stride_b % group_size != 0 || out_stride_h % group_size != 0)
        return SQUAT_ERR_SHAPE;
    if (batch == 0 || n_tokens == 0) return SQUAT_OK;
    if (s->lowrank_r > 0 && !s->prefer_dense)
        return squat_launch_quant_keys_lowrank(s->lr_table, k, dtype, batch, n_kv_heads, n_tokens, stride_b, stride_h, stride_t,
                                               bits, group_size, codes, scales, zeros, out_stride_b, out_stride_h, s->status,
                                               meta16, static_cast<cudaStream_t>(stream));
    return squat_launch_quant_keys(s->Wimg, k, dtype, batch, n_kv_heads, n_tokens, stride_b, stride_h, stride_t, bits,
                                   group_size, codes, scales, zeros, out_stride_b, out_stride_h, s->status, s->exact_blocks,
                                   meta16, static_cast<cudaStream_t>(stream));
}
}  // namespace

int squat_quantize_keys(const squat_subspace *s, const void *k, int dtype, int batch, int n_kv_heads,
                        int n_tokens, int head_dim, long long stride_b, long long stride_h,
                        long long stride_t, int bits, int group_size, unsigned char *codes,
                        float *scales, float *zeros, long long out_stride_b, long long out_stride_h,
                        void *stream)
{
    return quantize_keys_impl(s, k, dtype, batch, n_kv_heads, n_tokens, head_dim, stride_b, stride_h, stride_t, bits,
                              group_size, codes, scales, zeros, out_stride_b, out_stride_h, 0, stream);
}

int squat_quantize_keys_m16(const squat_subspace *s, const void *k, int dtype, int batch, int n_kv_heads,
                            int n_tokens, int head_dim, long long stride_b, long long stride_h,
                            long long stride_t, int bits, int group_size, unsigned char *codes,
                            void *scales, void *zeros, long long out_stride_b, long long out_stride_h,
                            void *stream)
{
    return quantize_keys_impl(s, k, dtype, batch, n_kv_heads, n_tokens, head_dim, stride_b, stride_h, stride_t, bits,
                              group_size, codes, scales, zeros, out_stride_b, out_stride_h, 1, stream);
}

namespace {
int quantize_values_impl(const void *v, int dtype, int batch, int n_kv_heads, int n_tokens,
                         int head_dim, long long stride_b, long long stride_h, long long stride_t,
                         int bits, int group_size, unsigned char *codes, void *scales, void *zeros,
                         long long out_stride_b, long long out_stride_h, int meta16, void *stream)
{
    int rc = check_quant_args(v, dtype, batch, n_kv_heads, n_tokens, head_dim, stride_b, stride_h, stride_t, bits,
                              group_size, codes, scales, zeros, out_stride_b, out_stride_h);
    if (rc != SQUAT_OK) return rc;
    if (head_dim % group_size != 0 || (head_dim * bits) % 64 != 0) return SQUAT_ERR_SHAPE;
    if (batch == 0 || n_tokens == 0) return SQUAT_OK;
    unsigned *status = squat_status_word();
    if (!status) return SQUAT_ERR_CUDA;
    return squat_launch_quant_values(v, dtype, batch, n_kv_heads, n_tokens, head_dim, stride_b, stride_h, stride_t,
                                     bits, group_size, codes, scales, zeros, out_stride_b, out_stride_h, status, meta16,
                                     static_cast<cudaStream_t>(stream));
}

int dequantize_impl(int kind, const unsigned char *codes, const void *scales, const void *zeros,
                    int batch, int n_kv_heads, int n_tokens, int head_dim, int bits, int group_size,
                    long long in_stride_b, long long in_stride_h, void *out, int out_dtype, int meta16, void *stream)
{
    if (!valid_dtype(out_dtype) || (kind != SQUAT_KEYS && kind != SQUAT_VALUES)) return SQUAT_ERR_INVALID_ARG;
    if (batch != 0 && n_tokens != 0 && (!codes || !scales || !zeros || !out)) return SQUAT_ERR_INVALID_ARG;
    if (!aligned16(codes) || !aligned16(scales) || !aligned16(zeros) || !aligned16(out)) return SQUAT_ERR_INVALID_ARG;
    if (batch < 0 || n_kv_heads <= 0 || n_tokens < 0 || head_dim <= 0 || in_stride_b < 0 || in_stride_h < 0)
        return SQUAT_ERR_INVALID_ARG;
    if (bits != 2 && bits != 4) return SQUAT_ERR_UNSUPPORTED;
    if (group_size != 32 && group_size != 64 && group_size != 128) return SQUAT_ERR_UNSUPPORTED;
    if (head_dim % 16 != 0) return SQUAT_ERR_SHAPE;
    if (kind == SQUAT_KEYS && (n_tokens % group_size || in_stride_b % group_size || in_stride_h % group_size))
        return SQUAT_ERR_SHAPE;
    if (kind == SQUAT_VALUES && head_dim % group_size) return SQUAT_ERR_SHAPE;
    return squat_launch_dequant(kind, codes, scales, zeros, batch, n_kv_heads, n_tokens, head_dim, bits, group_size,
                                in_stride_b, in_stride_h, out, out_dtype, meta16, static_cast<cudaStream_t>(stream));
}
}  // namespace

int squat_quantize_values(const void *v, int dtype, int batch, int n_kv_heads, int n_tokens,
                          int head_dim, long long stride_b, long long stride_h, long long stride_t,
                          int bits, int group_size, unsigned char *codes, float *scales, float *zeros,
                          long long out_stride_b, long long out_stride_h, void *stream)
{
    return quantize_values_impl(v, dtype, batch, n_kv_heads, n_tokens, head_dim, stride_b, stride_h, stride_t, bits,
                                group_size, codes, scales, zeros, out_stride_b, out_stride_h, 0, stream);
}

int squat_quantize_values_m16(const void *v, int dtype, int batch, int n_kv_heads, int n_tokens,
                              int head_dim, long long stride_b, long long stride_h, long long stride_t,
                              int bits, int group_size, unsigned char *codes, void *scales, void *zeros,
                              long long out_stride_b, long long out_stride_h, void *stream)
{
    return quantize_values_impl(v, dtype, batch, n_kv_heads, n_tokens, head_dim, stride_b, stride_h, stride_t, bits,
                                group_size, codes, scales, zeros, out_stride_b, out_stride_h, 1, stream);
}

int squat_dequantize(int kind, const unsigned char *codes, const float *scales, const float *zeros,
                     int batch, int n_kv_heads, int n_tokens, int head_dim, int bits, int group_size,
                     long long in_stride_b, long long in_stride_h, void *out, int out_dtype, void *stream)
{
    return dequantize_impl(kind, codes, scales, zeros, batch, n_kv_heads, n_tokens, head_dim, bits, group_size,
                           in_stride_b, in_stride_h, out, out_dtype, 0, stream);
}

int squat_dequantize_m16(int kind, const unsigned char *codes, const void *scales, const void *zeros,
                         int batch, int n_kv_heads, int n_tokens, int head_dim, int bits, int group_size,
                         long long in_stride_b, long long in_stride_h, void *out, int out_dtype, void *stream)
{
    return dequantize_impl(kind, codes, scales, zeros, batch, n_kv_heads, n_tokens, head_dim, bits, group_size,
                           in_stride_b, in_stride_h, out, out_dtype, 1, stream);
}

size_t squat_decode_attention_workspace_bytes(int batch, int n_q_heads, int n_tokens)
{
    if (batch <= 0 || n_q_heads <= 0 || n_tokens < 0) return 0;
    return (squat_attention_workspace_floats(batch, n_q_heads, n_tokens) * sizeof(float) + 255) / 256 * 256 + 256;
}

namespace {
int decode_attention_impl(const void *q, int q_dtype, int batch, int n_q_heads, int n_kv_heads, int head_dim,
                          const unsigned char *k_codes, const void *k_scales, const void *k_zeros,
                          const unsigned char *v_codes, const void *v_scales, const void *v_zeros,
                          int n_tokens, long long cache_stride_b, long long cache_stride_h, int bits,
                          int group_size, const void *k_res, const void *v_res, int res_dtype, int n_res,
                          float softmax_scale, float *out, void *workspace, size_t workspace_bytes,
                          const float *rope_table, int rope_blocks, long long first_pos, int meta16, void *stream)
{
    if (!valid_dtype(q_dtype) || batch < 0 || n_q_heads <= 0 || n_kv_heads <= 0 || n_tokens < 0 || n_res < 0)
        return SQUAT_ERR_INVALID_ARG;
    if (batch == 0) return SQUAT_OK;
    if (!q || !out || !workspace || !aligned16(q) || !aligned16(out)) return SQUAT_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return SQUAT_ERR_INVALID_ARG;
    if (head_dim != D || n_q_heads % n_kv_heads != 0) return SQUAT_ERR_SHAPE;
    if (bits != 2 && bits != 4) return SQUAT_ERR_UNSUPPORTED;
    if (group_size != 32 && group_size != 64 && group_size != 128) return SQUAT_ERR_UNSUPPORTED;
    if (n_res > SQUAT_ATTN_MAX_RESIDUAL) return SQUAT_ERR_UNSUPPORTED;
    if (n_tokens + n_res < 1) return SQUAT_ERR_SHAPE;
    if (n_tokens % group_size || cache_stride_b % group_size || cache_stride_h % group_size || cache_stride_b < 0 ||
        cache_stride_h < 0)
        return SQUAT_ERR_SHAPE;
    if (n_tokens > 0 && (!k_codes || !k_scales || !k_zeros || !v_codes || !v_scales || !v_zeros)) return SQUAT_ERR_INVALID_ARG;
    if (n_tokens > 0 && (!aligned16(k_codes) || !aligned16(k_scales) || !aligned16(k_zeros) || !aligned16(v_codes) ||
                         !aligned16(v_scales) || !aligned16(v_zeros)))
        return SQUAT_ERR_INVALID_ARG;
    if (n_res > 0 && (!k_res || !v_res || !valid_dtype(res_dtype) || !aligned16(k_res) || !aligned16(v_res)))
        return SQUAT_ERR_INVALID_ARG;
    if (workspace_bytes < squat_decode_attention_workspace_bytes(batch, n_q_heads, n_tokens)) return SQUAT_ERR_INVALID_ARG;
    const float scale = softmax_scale != 0.0f ? softmax_scale : 1.0f / sqrtf((float)head_dim);
    return squat_launch_decode_attention(q, q_dtype, batch, n_q_heads, n_kv_heads, n_tokens, k_codes, k_scales, k_zeros,
                                         v_codes, v_scales, v_zeros, cache_stride_b, cache_stride_h, bits, group_size,
                                         k_res, v_res, res_dtype, n_res, scale, out, static_cast<float *>(workspace),
                                         rope_table, rope_blocks, first_pos, meta16, static_cast<cudaStream_t>(stream));
}
}  // namespace

int squat_decode_attention(const void *q, int q_dtype, int batch, int n_q_heads, int n_kv_heads, int head_dim,
                           const unsigned char *k_codes, const float *k_scales, const float *k_zeros,
                           const unsigned char *v_codes, const float *v_scales, const float *v_zeros,
                           int n_tokens, long long cache_stride_b, long long cache_stride_h, int bits,
                           int group_size, const void *k_res, const void *v_res, int res_dtype, int n_res,
                           float softmax_scale, float *out, void *workspace, size_t workspace_bytes, void *stream)
{
    return decode_attention_impl(q, q_dtype, batch, n_q_heads, n_kv_heads, head_dim, k_codes, k_scales, k_zeros, v_codes,
                                 v_scales, v_zeros, n_tokens, cache_stride_b, cache_stride_h, bits, group_size, k_res, v_res,
                                 res_dtype, n_res, softmax_scale, out, workspace, workspace_bytes, nullptr, 0, 0, 0, stream);
}

int squat_decode_attention_ex(const void *q, int q_dtype, int batch, int n_q_heads, int n_kv_heads, int head_dim,
                              const unsigned char *k_codes, const void *k_scales, const void *k_zeros,
                              const unsigned char *v_codes, const void *v_scales, const void *v_zeros, int meta16,
                              int n_tokens, long long cache_stride_b, long long cache_stride_h, int bits,
                              int group_size, const void *k_res, const void *v_res, int res_dtype, int n_res,
                              float softmax_scale, const float *rope_table, int table_positions, long long first_pos,
                              float *out, void *workspace, size_t workspace_bytes, void *stream)
{
    if (meta16 != 0 && meta16 != 1) return SQUAT_ERR_INVALID_ARG;
    if (rope_table) {
        if (table_positions <= 0 || first_pos < 0 || n_tokens < 0 || n_res < 0 || !aligned16(rope_table)) return SQUAT_ERR_INVALID_ARG;
        if (first_pos % 32 != 0 || first_pos + n_tokens + n_res > table_positions) return SQUAT_ERR_SHAPE;
    }
    return decode_attention_impl(q, q_dtype, batch, n_q_heads, n_kv_heads, head_dim, k_codes, k_scales, k_zeros, v_codes,
                                 v_scales, v_zeros, n_tokens, cache_stride_b, cache_stride_h, bits, group_size, k_res, v_res,
                                 res_dtype, n_res, softmax_scale, out, workspace, workspace_bytes, rope_table,
                                 rope_table ? (table_positions + 31) / 32 : 0, first_pos, meta16, stream);
}

size_t squat_rope_table_floats(int n_positions)
{
    if (n_positions <= 0) return 0;
    return ((size_t)(n_positions + 31) / 32 + 32) * 64 * 2;
}

int squat_rope_table_fill(double base, int head_dim, int n_positions, float *table_host)
{
    if (!table_host || n_positions <= 0 || !(base > 0.0)) return SQUAT_ERR_INVALID_ARG;
    if (head_dim != D) return SQUAT_ERR_UNSUPPORTED;
    const int nb = (n_positions + 31) / 32, half = D / 2;
    for (int part = 0; part < 2; ++part) {
        const int rows = part == 0 ? nb : 32;
        float *t = table_host + (part == 0 ? 0 : (size_t)nb * half * 2);
        for (int r = 0; r < rows; ++r)
            for (int i = 0; i < half; ++i) {
                const double pos = part == 0 ? 32.0 * r : (double)r;
                const double a = pos * std::pow(base, -2.0 * i / (double)D);
                t[((size_t)r * half + i) * 2] = (float)std::cos(a);
                t[((size_t)r * half + i) * 2 + 1] = (float)std::sin(a);
            }
    }
    return SQUAT_OK;
}

int squat_decode_attention_pre_rope(const void *q, int q_dtype, int batch, int n_q_heads, int n_kv_heads, int head_dim,
                                    const unsigned char *k_codes, const float *k_scales, const float *k_zeros,
                                    const unsigned char *v_codes, const float *v_scales, const float *v_zeros,
                                    int n_tokens, long long cache_stride_b, long long cache_stride_h, int bits,
                                    int group_size, const void *k_res, const void *v_res, int res_dtype, int n_res,
                                    float softmax_scale, const float *rope_table, int table_positions,
                                    long long first_pos, float *out, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!rope_table || table_positions <= 0 || first_pos < 0 || n_tokens < 0 || n_res < 0) return SQUAT_ERR_INVALID_ARG;
    if (!aligned16(rope_table)) return SQUAT_ERR_INVALID_ARG;
    if (first_pos % 32 != 0) return SQUAT_ERR_SHAPE;
    if (first_pos + n_tokens + n_res > table_positions) return SQUAT_ERR_SHAPE;
    return decode_attention_impl(q, q_dtype, batch, n_q_heads, n_kv_heads, head_dim, k_codes, k_scales, k_zeros, v_codes,
                                 v_scales, v_zeros, n_tokens, cache_stride_b, cache_stride_h, bits, group_size, k_res, v_res,
                                 res_dtype, n_res, softmax_scale, out, workspace, workspace_bytes, rope_table,
                                 (table_positions + 31) / 32, first_pos, 0, stream);
}

#ifdef SQUAT_CHECKED
namespace {
// forms one address just inside and one just outside an extent; touches neither
__global__ void checked_selftest_kernel(const char *base, unsigned long long bytes, unsigned *status, int *passed_inside)
{
    SqExtent ext = {base, bytes};
    *passed_inside = SQ_CHK_G(status, base + bytes - 4, 4, ext) ? 1 : 0;      // last word: allowed, no flag
    (void)SQ_CHK_G(status, base + bytes - 3, 4, ext);                          // one byte over: refused, SQUAT_FLAG_BOUNDS
}
}  // namespace
#endif

int squat_checked_selftest(void *stream, int *detected)
{
#ifdef SQUAT_CHECKED
    if (!detected) return SQUAT_ERR_INVALID_ARG;
    unsigned *w = squat_status_word();
    if (!w) return SQUAT_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int *flag_dev = nullptr;
    unsigned before = 0, after = 0;
    int inside = 0;
    SQUAT_CUDA(cudaMalloc(&flag_dev, 256));
    SQUAT_CUDA(cudaMemcpyAsync(&before, w, sizeof(unsigned), cudaMemcpyDeviceToHost, st));
    SQUAT_CUDA(cudaStreamSynchronize(st));
    SQUAT_CUDA(cudaMemsetAsync(w, 0, sizeof(unsigned), st));
    checked_selftest_kernel<<<1, 1, 0, st>>>(reinterpret_cast<const char *>(flag_dev), 256, w, flag_dev);
    SQUAT_CUDA(cudaMemcpyAsync(&after, w, sizeof(unsigned), cudaMemcpyDeviceToHost, st));
    SQUAT_CUDA(cudaMemcpyAsync(&inside, flag_dev, sizeof(int), cudaMemcpyDeviceToHost, st));
    SQUAT_CUDA(cudaMemcpyAsync(w, &before, sizeof(unsigned), cudaMemcpyHostToDevice, st));      // the caller's flags are kept
    SQUAT_CUDA(cudaStreamSynchronize(st));
    cudaFree(flag_dev);
    *detected = (inside == 1 && (after & SQUAT_FLAG_BOUNDS)) ? 1 : 0;
    return SQUAT_OK;
#else
    (void)stream;
    if (detected) *detected = 0;
    return SQUAT_ERR_UNSUPPORTED;           // this is not the bounds-checked build
#endif
}

int squat_get_device_status(void *stream, unsigned *flags, int clear)
{
    if (!flags) return SQUAT_ERR_INVALID_ARG;
    unsigned *w = squat_status_word();
    if (!w) return SQUAT_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SQUAT_CUDA(cudaMemcpyAsync(flags, w, sizeof(unsigned), cudaMemcpyDeviceToHost, st));
    if (clear) SQUAT_CUDA(cudaMemsetAsync(w, 0, sizeof(unsigned), st));
    SQUAT_CUDA(cudaStreamSynchronize(st));
    return SQUAT_OK;
}

// ---------------------------------------------------------------------------------------
// Whole write path from host buffers.
namespace {
struct HostPathLayout {
    size_t q, k, v, kc, ks, kz, vc, vs, vz, x0, total;
};
HostPathLayout host_layout(int dtype, int batch, int n_q, int H, int T, int d, int bits, int G)
{
    HostPathLayout L;
    size_t off = 0;
    auto carve = [&](size_t bytes) { size_t o = off; off += (bytes + 255) / 256 * 256; return o; };
    const size_t es = elem_size(dtype);
    const size_t toks = (size_t)batch * H * T;
    L.q = carve((size_t)n_q * T * d * es);
    L.k = carve(toks * d * es);
    L.v = carve(toks * d * es);
    L.kc = carve(toks * d * bits / 8);
    L.ks = carve(toks / G * d * sizeof(float));
    L.kz = carve(toks / G * d * sizeof(float));
    L.vc = carve(toks * d * bits / 8);
    L.vs = carve(toks * (d / G) * sizeof(float));
    L.vz = carve(toks * (d / G) * sizeof(float));
    L.x0 = carve((size_t)D * 64 * sizeof(double));     // start block of the block power build (rank <= 64)
    L.total = off;
    return L;
}
}  // namespace

size_t squat_write_path_workspace_bytes(int dtype, int batch, int n_q_heads, int n_kv_heads,
                                        int n_tokens, int head_dim, int bits, int group_size)
{
    if (!valid_dtype(dtype) || batch <= 0 || n_q_heads <= 0 || n_kv_heads <= 0 || n_tokens <= 0 || head_dim <= 0 ||
        (bits != 2 && bits != 4) || group_size <= 0)
        return 0;
    return host_layout(dtype, batch, n_q_heads, n_kv_heads, n_tokens, head_dim, bits, group_size).total;
}

}  // extern "C"

namespace {
int write_path_host_impl(squat_subspace *s, const void *q_host, const void *k_host, const void *v_host,
                         int dtype, int batch, int n_q_heads, int n_kv_heads, int n_tokens,
                         int head_dim, int rank_r, double lambda, int block_g, int bits, int group_size,
                         unsigned char *k_codes_host, void *k_scales_host, void *k_zeros_host,
                         unsigned char *v_codes_host, void *v_scales_host, void *v_zeros_host,
                         int meta16, const double *start_block_host, int power_iters,
                         void *workspace, size_t workspace_bytes, void *stream)
{
    // q_host == NULL: no build; the keys are quantized with the update matrices the handle already holds (a decode window)
    const bool do_build = q_host != nullptr;
    if (!s || !k_host || !v_host || !k_codes_host || !k_scales_host || !k_zeros_host || !v_codes_host ||
        !v_scales_host || !v_zeros_host || !workspace || !valid_dtype(dtype))
        return SQUAT_ERR_INVALID_ARG;
    if (!on_handle_device(s)) return SQUAT_ERR_INVALID_ARG;     // the handle belongs to another device
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return SQUAT_ERR_INVALID_ARG;
    if (batch <= 0 || n_tokens <= 0 || head_dim != D || n_kv_heads != s->n_kv_heads) return SQUAT_ERR_SHAPE;
    if ((bits != 2 && bits != 4) || (group_size != 32 && group_size != 64 && group_size != 128))
        return SQUAT_ERR_UNSUPPORTED;
    if (n_tokens % group_size) return SQUAT_ERR_SHAPE;
    const HostPathLayout L = host_layout(dtype, batch, n_q_heads, n_kv_heads, n_tokens, head_dim, bits, group_size);
    if (workspace_bytes < L.total) return SQUAT_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char *w = static_cast<char *>(workspace);
    const size_t es = elem_size(dtype);
    const size_t toks = (size_t)batch * n_kv_heads * n_tokens;
    const long long T = n_tokens, d = head_dim;
    const size_t ms = meta16 ? 2 : sizeof(float);          // bytes per stored scale / zero-point
    if (start_block_host && (rank_r < 0 || rank_r > 64)) return rank_r < 0 ? SQUAT_ERR_INVALID_ARG : SQUAT_ERR_UNSUPPORTED;
    // Copies and kernels overlap: q goes up first (the subspace build needs it), k and v follow on a side stream
    // while the build runs; the key outputs go down on a second side stream while v is still coming up.  v travels
    // in up to four pieces ((batch, head) ranges): each is quantized and its outputs sent down as soon as it has
    // arrived, so that only the last piece's kernel and download are left when the upload ends.  Everything is
    // ordered after the work already in `stream` and joined back into it.
    if (!s->side_ready) {
        for (int i = 0; i < 2; ++i) SQUAT_CUDA(cudaStreamCreateWithFlags(&s->side[i], cudaStreamNonBlocking));
        for (int i = 0; i < 8; ++i) SQUAT_CUDA(cudaEventCreateWithFlags(&s->ev[i], cudaEventDisableTiming));
        s->side_ready = true;
    }
    cudaEvent_t ev_q = s->ev[0], ev_k = s->ev[1], ev_keys = s->ev[2], ev_kout = s->ev[3];
    const long long rows = (long long)batch * n_kv_heads;          // (batch, head) units of T tokens
    const int n_pieces = rows >= 4 ? 4 : (int)rows;
    if (do_build) SQUAT_CUDA(cudaMemcpyAsync(w + L.q, q_host, (size_t)n_q_heads * T * d * es, cudaMemcpyHostToDevice, st));
    if (do_build && start_block_host && rank_r > 0)
        SQUAT_CUDA(cudaMemcpyAsync(w + L.x0, start_block_host, (size_t)D * rank_r * sizeof(double), cudaMemcpyHostToDevice, st));
    SQUAT_CUDA(cudaEventRecord(ev_q, st));
    SQUAT_CUDA(cudaStreamWaitEvent(s->side[0], ev_q, 0));
    SQUAT_CUDA(cudaMemcpyAsync(w + L.k, k_host, toks * d * es, cudaMemcpyHostToDevice, s->side[0]));
    SQUAT_CUDA(cudaEventRecord(ev_k, s->side[0]));
    for (int p = 0; p < n_pieces; ++p) {
        const long long r0 = rows * p / n_pieces, r1 = rows * (p + 1) / n_pieces;
        SQUAT_CUDA(cudaMemcpyAsync(w + L.v + (size_t)r0 * T * d * es, static_cast<const char *>(v_host) + (size_t)r0 * T * d * es,
                                   (size_t)(r1 - r0) * T * d * es, cudaMemcpyHostToDevice, s->side[0]));
        SQUAT_CUDA(cudaEventRecord(s->ev[4 + p], s->side[0]));
    }
    int rc = SQUAT_OK;
    if (do_build)
        rc = start_block_host
                 ? squat_build_subspace_power(s, w + L.q, dtype, n_q_heads, n_tokens, T * d, d, rank_r, lambda, block_g,
                                              reinterpret_cast<const double *>(w + L.x0), 0, power_iters, stream)
                 : squat_build_subspace(s, w + L.q, dtype, n_q_heads, n_tokens, T * d, d, rank_r, lambda, block_g, stream);
    if (rc != SQUAT_OK) return rc;
    SQUAT_CUDA(cudaStreamWaitEvent(st, ev_k, 0));
    rc = quantize_keys_impl(s, w + L.k, dtype, batch, n_kv_heads, n_tokens, head_dim, (long long)n_kv_heads * T * d,
                            T * d, d, bits, group_size, reinterpret_cast<unsigned char *>(w + L.kc),
                            w + L.ks, w + L.kz, (long long)n_kv_heads * T, T, meta16, stream);
    if (rc != SQUAT_OK) return rc;
    SQUAT_CUDA(cudaEventRecord(ev_keys, st));
    SQUAT_CUDA(cudaStreamWaitEvent(s->side[1], ev_keys, 0));
    SQUAT_CUDA(cudaMemcpyAsync(k_codes_host, w + L.kc, toks * d * bits / 8, cudaMemcpyDeviceToHost, s->side[1]));
    SQUAT_CUDA(cudaMemcpyAsync(k_scales_host, w + L.ks, toks / group_size * d * ms, cudaMemcpyDeviceToHost, s->side[1]));
    SQUAT_CUDA(cudaMemcpyAsync(k_zeros_host, w + L.kz, toks / group_size * d * ms, cudaMemcpyDeviceToHost, s->side[1]));
    SQUAT_CUDA(cudaEventRecord(ev_kout, s->side[1]));
    const size_t vrow_codes = (size_t)T * d * bits / 8, vrow_meta = (size_t)T * (d / group_size) * ms;
    for (int p = 0; p < n_pieces; ++p) {
        const long long r0 = rows * p / n_pieces, r1 = rows * (p + 1) / n_pieces;
        SQUAT_CUDA(cudaStreamWaitEvent(st, s->ev[4 + p], 0));
        rc = quantize_values_impl(w + L.v + (size_t)r0 * T * d * es, dtype, 1, (int)(r1 - r0), n_tokens, head_dim, 0, T * d, d,
                                  bits, group_size, reinterpret_cast<unsigned char *>(w + L.vc) + r0 * vrow_codes,
                                  w + L.vs + r0 * vrow_meta, w + L.vz + r0 * vrow_meta, 0, T, meta16, stream);
        if (rc != SQUAT_OK) return rc;
        SQUAT_CUDA(cudaMemcpyAsync(v_codes_host + r0 * vrow_codes, w + L.vc + r0 * vrow_codes, (r1 - r0) * vrow_codes, cudaMemcpyDeviceToHost, st));
        SQUAT_CUDA(cudaMemcpyAsync(static_cast<char *>(v_scales_host) + r0 * vrow_meta, w + L.vs + r0 * vrow_meta, (r1 - r0) * vrow_meta, cudaMemcpyDeviceToHost, st));
        SQUAT_CUDA(cudaMemcpyAsync(static_cast<char *>(v_zeros_host) + r0 * vrow_meta, w + L.vz + r0 * vrow_meta, (r1 - r0) * vrow_meta, cudaMemcpyDeviceToHost, st));
    }
    SQUAT_CUDA(cudaStreamWaitEvent(st, ev_kout, 0));
    SQUAT_CUDA(cudaStreamSynchronize(st));
    return SQUAT_OK;
}
}  // namespace

extern "C" {

int squat_write_path_host(squat_subspace *s, const void *q_host, const void *k_host, const void *v_host,
                          int dtype, int batch, int n_q_heads, int n_kv_heads, int n_tokens,
                          int head_dim, int rank_r, double lambda, int block_g, int bits, int group_size,
                          unsigned char *k_codes_host, float *k_scales_host, float *k_zeros_host,
                          unsigned char *v_codes_host, float *v_scales_host, float *v_zeros_host,
                          void *workspace, size_t workspace_bytes, void *stream)
{
    if (!q_host) return SQUAT_ERR_INVALID_ARG;
    return write_path_host_impl(s, q_host, k_host, v_host, dtype, batch, n_q_heads, n_kv_heads, n_tokens, head_dim, rank_r,
                                lambda, block_g, bits, group_size, k_codes_host, k_scales_host, k_zeros_host, v_codes_host,
                                v_scales_host, v_zeros_host, 0, nullptr, 0, workspace, workspace_bytes, stream);
}

int squat_append_window_host(squat_subspace *s, const void *k_host, const void *v_host, int dtype, int batch,
                             int n_kv_heads, int n_tokens, int head_dim, int bits, int group_size,
                             unsigned char *k_codes_host, void *k_scales_host, void *k_zeros_host,
                             unsigned char *v_codes_host, void *v_scales_host, void *v_zeros_host, int meta16,
                             void *workspace, size_t workspace_bytes, void *stream)
{
    if (meta16 != 0 && meta16 != 1) return SQUAT_ERR_INVALID_ARG;
    return write_path_host_impl(s, nullptr, k_host, v_host, dtype, batch, n_kv_heads, n_kv_heads, n_tokens, head_dim, 0, 0.0, 1,
                                bits, group_size, k_codes_host, k_scales_host, k_zeros_host, v_codes_host, v_scales_host,
                                v_zeros_host, meta16, nullptr, 0, workspace, workspace_bytes, stream);
}

int squat_write_path_host_ex(squat_subspace *s, const void *q_host, const void *k_host, const void *v_host,
                             int dtype, int batch, int n_q_heads, int n_kv_heads, int n_tokens,
                             int head_dim, int rank_r, double lambda, int block_g, int bits, int group_size,
                             unsigned char *k_codes_host, void *k_scales_host, void *k_zeros_host,
                             unsigned char *v_codes_host, void *v_scales_host, void *v_zeros_host,
                             int meta16, const double *start_block_host, int power_iters,
                             void *workspace, size_t workspace_bytes, void *stream)
{
    if (meta16 != 0 && meta16 != 1) return SQUAT_ERR_INVALID_ARG;
    if (!q_host) return SQUAT_ERR_INVALID_ARG;
    return write_path_host_impl(s, q_host, k_host, v_host, dtype, batch, n_q_heads, n_kv_heads, n_tokens, head_dim, rank_r,
                                lambda, block_g, bits, group_size, k_codes_host, k_scales_host, k_zeros_host, v_codes_host,
                                v_scales_host, v_zeros_host, meta16, start_block_host, power_iters, workspace,
                                workspace_bytes, stream);
}

}  // extern "C"
