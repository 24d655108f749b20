// Internal helpers shared by the CUDA translation units of libchela (not part of the C ABI).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "chela.h"

namespace chela {

inline chela_status_t cuda_status(cudaError_t e) { return e == cudaSuccess ? CHELA_OK : CHELA_ERR_CUDA; }
inline chela_status_t last_launch_status() { return cuda_status(cudaGetLastError()); }

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int next_pow2(int x) { int p = 1; while (p < x) p <<= 1; return p; }
inline size_t dtype_size(chela_dtype_t t) { return t == CHELA_F32 ? 4 : (t == CHELA_BF16 ? 2 : 4); }  // pair: two bf16 planes
inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

__device__ __forceinline__ float silu_f(float u) { return u / (1.0f + __expf(-u)); }
__device__ __forceinline__ float sigmoid_f(float u) { return 1.0f / (1.0f + __expf(-u)); }
// activation codes of the dense kernels: 0 identity, 1 SiLU, 2 sigmoid
__device__ __forceinline__ float activate(float u, int act) { return act == 1 ? silu_f(u) : (act == 2 ? sigmoid_f(u) : u); }

// Load / store 4 consecutive elements as fp32.
__device__ __forceinline__ float4 load4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16 *p)
{
    uint2 u = *reinterpret_cast<const uint2 *>(p);
    __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162 *>(&u.x);
    __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162 *>(&u.y);
    float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
    return make_float4(fa.x, fa.y, fb.x, fb.y);
}
__device__ __forceinline__ void store4(float *p, float4 v) { *reinterpret_cast<float4 *>(p) = v; }
__device__ __forceinline__ void store4(__nv_bfloat16 *p, float4 v)
{
    __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
    uint2 u;
    u.x = *reinterpret_cast<uint32_t *>(&a);
    u.y = *reinterpret_cast<uint32_t *>(&b);
    *reinterpret_cast<uint2 *>(p) = u;
}
__device__ __forceinline__ float load1(const float *p) { return *p; }
__device__ __forceinline__ float load1(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
__device__ __forceinline__ void store1(float *p, float v) { *p = v; }
__device__ __forceinline__ void store1(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

// How long a device-side wait may last, and the test hook that makes one run out: the tensor-core kernels take this
// by value.  `limit` is in SM cycles; `skip_arrival` != 0 asks CTA 0 to leave out one mbarrier arrival (the role that
// waits for it then gives up after `limit` cycles, records CHELA_ERR_TIMEOUT and the kernel returns by itself).
struct WaitCtl {
    long long limit;
    int skip_arrival;
};
WaitCtl current_wait_ctl();   // what chela_debug_wait_control last set (default: about one second, no skipped arrival)

// ---- launchers implemented in the other translation units ------------------------------------

chela_status_t launch_linattn_simt(const void *q, const void *k, const void *v, void *o, int B, int H,
                                   int L, int d, int chunk, chela_dtype_t in_dtype,
                                   chela_dtype_t out_dtype, int norm, float eps, float scale,
                                   cudaStream_t stream, const float *state_in = nullptr, float *state_out = nullptr);

// tcgen05/TMEM/TMA kernel for bf16 inputs
bool linattn_sm100_supported(int B, int H, int L, int d, int chunk, chela_dtype_t in_dtype,
                             chela_dtype_t out_dtype);
size_t linattn_sm100_workspace_bytes(int B, int H, int L, int d, int chunk);
chela_status_t launch_linattn_sm100(const void *q, const void *k, const void *v, void *o, int B, int H,
                                    int L, int d, int chunk, chela_dtype_t in_dtype,
                                    chela_dtype_t out_dtype, int norm, float eps, float scale,
                                    void *workspace, cudaStream_t stream, const float *state_in = nullptr,
                                    float *state_out = nullptr, bool reverse = false, int pair_mask = 7, bool keep_status = false);

// chain-free kernel for plain bf16, d = 64, fewer (batch, head) pairs than SMs (one CTA per SM, `stride` CTAs per sequence)
int linattn_sm100_pipe_stride(int B, int H, int L, int sms);
chela_status_t launch_linattn_sm100_pipe(const void *q, const void *k, const void *v, void *o, int B, int H, int L, int stride,
                                         chela_dtype_t out_dtype, int norm, float eps, float scale, int *status,
                                         const float *state_in, float *state_out, cudaStream_t stream);

size_t linattn_sm100_d128_workspace_bytes(int B, int H, int L);
void linattn_sm100_d128_split(int B, int H, int L, int sms, int *G, int *cg0, int *cg);
void linattn_sm100_split(int B, int H, int L, int d, bool full_pair, int sms, int *G, int *cg0, int *cg);
chela_status_t launch_linattn_sm100_d128(const void *q, const void *k, const void *v, void *o, int B, int H, int L,
                                         chela_dtype_t in_dtype, chela_dtype_t out_dtype, int norm, float eps, float scale,
                                         void *workspace, cudaStream_t stream, const float *state_in = nullptr,
                                         float *state_out = nullptr, bool reverse = false, int pair_mask = 7, bool keep_status = false);

// backward of causal linear attention (fp32 SIMT); gradients fp32; workspace = one [B,L,H,d] fp32 buffer
size_t linattn_bwd_workspace_bytes(int B, int H, int L, int d);
chela_status_t launch_linattn_bwd_simt(const void *q, const void *k, const void *v, const void *d_o, float *dq, float *dk,
                                       float *dv, int B, int H, int L, int d, chela_dtype_t in_dtype, int norm, float eps,
                                       float scale, void *workspace, cudaStream_t stream);

// tensor-core backward (bf16, d = 64): four launches of the forward kernel plus an elementwise kernel
chela_status_t launch_linattn_step(const void *q, const void *k, const void *v, void *o, float *state, int B, int H, int d,
                                   chela_dtype_t in_dtype, chela_dtype_t out_dtype, int norm, float eps, float scale,
                                   cudaStream_t stream);
chela_status_t launch_linattn_sm100_grad(const void *q, const void *k, const void *v, const void *d_o, void *g, int B, int H, int L,
                                         float eps, float scale, void *workspace, cudaStream_t stream);
bool linattn_bwd_sm100_supported(int d, chela_dtype_t in_dtype);
size_t linattn_bwd_sm100_workspace_bytes(int B, int H, int L, int d);
chela_status_t launch_linattn_bwd_sm100(const void *q, const void *k, const void *v, const void *d_o, float *dq, float *dk,
                                        float *dv, int B, int H, int L, int d, int norm, float eps, float scale,
                                        void *workspace, cudaStream_t stream);

chela_status_t launch_shortconv(const void *x, const float *w, const float *bias, void *y, int B, int L,
                                int D, int width, int act, chela_dtype_t io_dtype, cudaStream_t stream);

chela_status_t launch_shortconv_reparam(const float *w1, int width1, const float *w2, int width2, float *merged, int D,
                                        cudaStream_t stream);

size_t longconv_workspace_bytes(int B, int L, int D);
bool launch_fft_conv_fast(int mode, float *rows, int row_stride, int L, int D, int nrows, int logM, const float2 *tw,
                          float2 *spec, int spec_stride, cudaStream_t stream, __nv_bfloat16 *zt = nullptr,
                          size_t zt_lo_offset = 0);
bool longconv_transposed_pair_supported(int L);
int longconv_row_stride(int L);
chela_status_t launch_longconv(const void *x, const float *k_long, const float *w_short, int short_width,
                               void *z, int B, int L, int D, chela_dtype_t in_dtype,
                               chela_dtype_t out_dtype, void *workspace, cudaStream_t stream, bool transposed_pair = false,
                               const void *spectrum = nullptr);
size_t longconv_spectrum_bytes(int L, int D);
chela_status_t launch_longconv_prepare(const float *k_long, int L, int D, void *spectrum, cudaStream_t stream);

// y[M,N] = act(a[M,K] w[K,N] + bias[N]); a: a_dtype, w: w_dtype, y: y_dtype.
chela_status_t launch_gemm_simt(const void *a, const void *w, const float *bias, void *y, size_t M, int K,
                                int N, int act, chela_dtype_t a_dtype, chela_dtype_t w_dtype,
                                chela_dtype_t y_dtype, cudaStream_t stream);
// tcgen05 GEMM: a bf16 or bf16 pair, w bf16, y bf16 or bf16 pair
bool gemm_sm100_supported(size_t M, int K, int N, chela_dtype_t a_dtype, chela_dtype_t w_dtype, chela_dtype_t y_dtype);
bool gemm_sm100_at_supported(int B, int L, int Ls, int K, int N);
chela_status_t launch_gemm_sm100_at(const void *at, int B, int L, int Ls, const void *w, const float *bias, void *y, int K, int N,
                                    int act, int *status, cudaStream_t stream);
chela_status_t launch_gemm_sm100(const void *a, const void *w, const float *bias, void *y, size_t M, int K, int N,
                                 int act, chela_dtype_t a_dtype, chela_dtype_t y_dtype, int *status, cudaStream_t stream);
// y[m,c] = alpha[c] * z[m,c] + beta[c]
chela_status_t launch_affine(const float *z, const void *alpha, const float *beta, float *y, size_t M, int D,
                             chela_dtype_t alpha_dtype, cudaStream_t stream);

// the same on bf16 pairs ([2][M*D] bf16 in and out)
chela_status_t launch_affine_pair(const void *z, const void *alpha, const float *beta, void *y, size_t M, int D,
                                  chela_dtype_t alpha_dtype, cudaStream_t stream);

// u = o * g_a * g_o + x * (1 - g_o)  (Eqs. 8, 14); o fp32, gates fp32 or bf16 pairs, x and u in their own dtypes
chela_status_t launch_gate_combine(const float *o, const void *g_a, const void *g_o, chela_dtype_t gate_dtype, const void *x,
                                   chela_dtype_t x_dtype, void *u, chela_dtype_t u_dtype, size_t n, cudaStream_t stream);

}  // namespace chela
