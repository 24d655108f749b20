// fp32 SIMT GEMM for the Q/K/V formation of the mixer (Eqs. 10-12): y = act(a w + bias).
// 128 x 128 x 16 tiles, 256 threads, 8 x 8 outputs per thread, fp32 FFMA accumulation.  It keeps
// the long-convolution output Z and the resulting Q, K in fp32, which the normalised mixer
// output needs (bf16 Q/K lose the result's leading digits to cancellation in Q K^T).
#include "common.cuh"

namespace chela {
namespace {

constexpr int BM = 128, BN = 128, BK = 16;

template <typename TA, typename TW, typename TY>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const TA *__restrict__ a, const TW *__restrict__ w, const float *__restrict__ bias,
                 TY *__restrict__ y, size_t M, int K, int N, int act)
{
    __shared__ float sA[BK][BM + 4];  // a tile transposed: [k][m]
    __shared__ float sW[BK][BN + 4];  // [k][n]
    const int tid = threadIdx.x;
    const size_t m0 = (size_t)blockIdx.y * BM;
    const int n0 = blockIdx.x * BN;
    const int tm = (tid / 16) * 8, tn = (tid % 16) * 8;
    float acc[8][8] = {};

    for (int k0 = 0; k0 < K; k0 += BK) {
        // a tile: 128 rows x 16 k; 2048 elements, 8 per thread
        for (int idx = tid; idx < BM * BK; idx += 256) {
            const int r = idx / BK, kk = idx % BK;
            const size_t m = m0 + r;
            sA[kk][r] = (m < M && k0 + kk < K) ? load1(a + m * K + k0 + kk) : 0.f;
        }
        for (int idx = tid; idx < BK * BN; idx += 256) {
            const int kk = idx / BN, c = idx % BN;
            sW[kk][c] = (k0 + kk < K && n0 + c < N) ? load1(w + (size_t)(k0 + kk) * N + n0 + c) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            const float4 a0 = load4(&sA[kk][tm]), a1 = load4(&sA[kk][tm + 4]);
            const float4 w0 = load4(&sW[kk][tn]), w1 = load4(&sW[kk][tn + 4]);
            const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const float wv[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(av[i], wv[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const size_t m = m0 + tm + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int n = n0 + tn + j;
            if (n >= N) continue;
            float r = acc[i][j] + (bias ? bias[n] : 0.f);
            if (act) r = activate(r, act);
            store1(y + m * N + n, r);
        }
    }
}

template <typename TA, typename TW, typename TY>
chela_status_t launch_t(const void *a, const void *w, const float *bias, void *y, size_t M, int K, int N,
                        int act, cudaStream_t stream)
{
    dim3 grid((N + BN - 1) / BN, (unsigned)((M + BM - 1) / BM));
    gemm_simt_kernel<TA, TW, TY><<<grid, 256, 0, stream>>>((const TA *)a, (const TW *)w, bias, (TY *)y, M, K, N, act);
    return last_launch_status();
}

template <typename TW>
__global__ void affine_kernel(const float *__restrict__ z, const TW *__restrict__ alpha,
                              const float *__restrict__ beta, float *__restrict__ y, size_t n, int D)
{
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % D);
        y[i] = fmaf(load1(alpha + c), z[i], beta ? beta[c] : 0.f);
    }
}

// bf16-pair version: z, y are [2][n] bf16 (high plane, low plane)
template <typename TW>
__global__ void affine_pair_kernel(const __nv_bfloat16 *__restrict__ z, const TW *__restrict__ alpha,
                                   const float *__restrict__ beta, __nv_bfloat16 *__restrict__ y, size_t n, int D)
{
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % D);
        const float v = fmaf(load1(alpha + c), __bfloat162float(z[i]) + __bfloat162float(z[n + i]), beta ? beta[c] : 0.f);
        const __nv_bfloat16 hi = __float2bfloat16_rn(v);
        y[i] = hi;
        y[n + i] = __float2bfloat16_rn(v - __bfloat162float(hi));
    }
}

}  // namespace

chela_status_t launch_affine_pair(const void *z, const void *alpha, const float *beta, void *y, size_t M, int D,
                                  chela_dtype_t alpha_dtype, cudaStream_t stream)
{
    const size_t n = M * D;
    const int blocks = (int)((n + 255) / 256 < 148 * 16 ? (n + 255) / 256 : 148 * 16);
    if (alpha_dtype == CHELA_BF16)
        affine_pair_kernel<__nv_bfloat16><<<blocks, 256, 0, stream>>>((const __nv_bfloat16 *)z, (const __nv_bfloat16 *)alpha, beta,
                                                                      (__nv_bfloat16 *)y, n, D);
    else
        affine_pair_kernel<float><<<blocks, 256, 0, stream>>>((const __nv_bfloat16 *)z, (const float *)alpha, beta,
                                                              (__nv_bfloat16 *)y, n, D);
    return last_launch_status();
}

namespace {
template <typename TG, typename TX, typename TU>
__global__ void gate_combine_kernel(const float *__restrict__ o, const TG *__restrict__ g_a, const TG *__restrict__ g_o,
                                    const TX *__restrict__ x, TU *__restrict__ u, size_t n, int pair)
{
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        float ga = load1(g_a + i), go = load1(g_o + i);
        if (pair) {   // bf16 pair: low plane n elements later
            ga += load1(g_a + n + i);
            go += load1(g_o + n + i);
        }
        store1(u + i, fmaf(o[i] * ga, go, load1(x + i) * (1.0f - go)));
    }
}
// The mixer's case, eight elements per thread with 16-byte accesses: bf16-pair gates, bf16 x, fp32 o and u.
__global__ void __launch_bounds__(256)
gate_combine_vec_kernel(const float *__restrict__ o, const __nv_bfloat16 *__restrict__ g_a, const __nv_bfloat16 *__restrict__ g_o,
                        const __nv_bfloat16 *__restrict__ x, float *__restrict__ u, size_t n)
{
    for (size_t i = (blockIdx.x * (size_t)blockDim.x + threadIdx.x) * 8; i < n; i += (size_t)gridDim.x * blockDim.x * 8) {
        const uint4 ah = *reinterpret_cast<const uint4 *>(g_a + i), al = *reinterpret_cast<const uint4 *>(g_a + n + i);
        const uint4 oh = *reinterpret_cast<const uint4 *>(g_o + i), ol = *reinterpret_cast<const uint4 *>(g_o + n + i);
        const uint4 xv = *reinterpret_cast<const uint4 *>(x + i);
        const float4 o0 = *reinterpret_cast<const float4 *>(o + i), o1 = *reinterpret_cast<const float4 *>(o + i + 4);
        const float ov[8] = {o0.x, o0.y, o0.z, o0.w, o1.x, o1.y, o1.z, o1.w};
        const __nv_bfloat162 *pah = reinterpret_cast<const __nv_bfloat162 *>(&ah), *pal = reinterpret_cast<const __nv_bfloat162 *>(&al);
        const __nv_bfloat162 *poh = reinterpret_cast<const __nv_bfloat162 *>(&oh), *pol = reinterpret_cast<const __nv_bfloat162 *>(&ol);
        const __nv_bfloat162 *px = reinterpret_cast<const __nv_bfloat162 *>(&xv);
        float r[8];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 a_h = __bfloat1622float2(pah[e]), a_l = __bfloat1622float2(pal[e]);
            const float2 g_h = __bfloat1622float2(poh[e]), g_l = __bfloat1622float2(pol[e]);
            const float2 xx = __bfloat1622float2(px[e]);
            const float ga0 = a_h.x + a_l.x, ga1 = a_h.y + a_l.y, go0 = g_h.x + g_l.x, go1 = g_h.y + g_l.y;
            r[2 * e] = fmaf(ov[2 * e] * ga0, go0, xx.x * (1.0f - go0));
            r[2 * e + 1] = fmaf(ov[2 * e + 1] * ga1, go1, xx.y * (1.0f - go1));
        }
        *reinterpret_cast<float4 *>(u + i) = make_float4(r[0], r[1], r[2], r[3]);
        *reinterpret_cast<float4 *>(u + i + 4) = make_float4(r[4], r[5], r[6], r[7]);
    }
}

template <typename TG>
chela_status_t gate_combine_t(const float *o, const void *g_a, const void *g_o, int pair, const void *x, chela_dtype_t x_dtype,
                              void *u, chela_dtype_t u_dtype, size_t n, cudaStream_t stream)
{
    typedef __nv_bfloat16 bf;
    const int blocks = (int)((n + 255) / 256 < 148 * 32 ? (n + 255) / 256 : 148 * 32);
    const TG *ga = (const TG *)g_a, *go = (const TG *)g_o;
    if (x_dtype == CHELA_BF16 && u_dtype == CHELA_BF16)
        gate_combine_kernel<TG, bf, bf><<<blocks, 256, 0, stream>>>(o, ga, go, (const bf *)x, (bf *)u, n, pair);
    else if (x_dtype == CHELA_BF16)
        gate_combine_kernel<TG, bf, float><<<blocks, 256, 0, stream>>>(o, ga, go, (const bf *)x, (float *)u, n, pair);
    else if (u_dtype == CHELA_BF16)
        gate_combine_kernel<TG, float, bf><<<blocks, 256, 0, stream>>>(o, ga, go, (const float *)x, (bf *)u, n, pair);
    else
        gate_combine_kernel<TG, float, float><<<blocks, 256, 0, stream>>>(o, ga, go, (const float *)x, (float *)u, n, pair);
    return last_launch_status();
}
}  // namespace

chela_status_t launch_gate_combine(const float *o, const void *g_a, const void *g_o, chela_dtype_t gate_dtype, const void *x,
                                   chela_dtype_t x_dtype, void *u, chela_dtype_t u_dtype, size_t n, cudaStream_t stream)
{
    if (gate_dtype == CHELA_BF16_PAIR && x_dtype == CHELA_BF16 && u_dtype == CHELA_F32 && n % 8 == 0) {
        const size_t threads = n / 8;
        const int blocks = (int)((threads + 255) / 256 < 148 * 16 ? (threads + 255) / 256 : 148 * 16);
        gate_combine_vec_kernel<<<blocks, 256, 0, stream>>>(o, (const __nv_bfloat16 *)g_a, (const __nv_bfloat16 *)g_o,
                                                            (const __nv_bfloat16 *)x, (float *)u, n);
        return last_launch_status();
    }
    if (gate_dtype == CHELA_BF16_PAIR) return gate_combine_t<__nv_bfloat16>(o, g_a, g_o, 1, x, x_dtype, u, u_dtype, n, stream);
    return gate_combine_t<float>(o, g_a, g_o, 0, x, x_dtype, u, u_dtype, n, stream);
}

chela_status_t launch_gemm_simt(const void *a, const void *w, const float *bias, void *y, size_t M, int K,
                                int N, int act, chela_dtype_t a_dtype, chela_dtype_t w_dtype,
                                chela_dtype_t y_dtype, cudaStream_t stream)
{
    typedef __nv_bfloat16 bf;
    const int key = (a_dtype == CHELA_BF16) * 4 + (w_dtype == CHELA_BF16) * 2 + (y_dtype == CHELA_BF16);
    switch (key) {
        case 0: return launch_t<float, float, float>(a, w, bias, y, M, K, N, act, stream);
        case 1: return launch_t<float, float, bf>(a, w, bias, y, M, K, N, act, stream);
        case 2: return launch_t<float, bf, float>(a, w, bias, y, M, K, N, act, stream);
        case 3: return launch_t<float, bf, bf>(a, w, bias, y, M, K, N, act, stream);
        case 4: return launch_t<bf, float, float>(a, w, bias, y, M, K, N, act, stream);
        case 5: return launch_t<bf, float, bf>(a, w, bias, y, M, K, N, act, stream);
        case 6: return launch_t<bf, bf, float>(a, w, bias, y, M, K, N, act, stream);
        default: return launch_t<bf, bf, bf>(a, w, bias, y, M, K, N, act, stream);
    }
}

chela_status_t launch_affine(const float *z, const void *alpha, const float *beta, float *y, size_t M, int D,
                             chela_dtype_t alpha_dtype, cudaStream_t stream)
{
    const size_t n = M * D;
    const int blocks = (int)((n + 255) / 256 < 148 * 16 ? (n + 255) / 256 : 148 * 16);
    if (alpha_dtype == CHELA_BF16)
        affine_kernel<__nv_bfloat16><<<blocks, 256, 0, stream>>>(z, (const __nv_bfloat16 *)alpha, beta, y, n, D);
    else
        affine_kernel<float><<<blocks, 256, 0, stream>>>(z, (const float *)alpha, beta, y, n, D);
    return last_launch_status();
}

}  // namespace chela
