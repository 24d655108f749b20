// Backward of chunked causal linear attention, fp32 SIMT kernel (gradients of Eq. 2 with the causal mask
// and the row normaliser, evaluated with the tiling of Sec. 4.1 in both directions).
//
// With G_t = scale * dLoss/dr_t (the output gradient pulled back through the normaliser):
//   forward sweep  (running state S = sum K^T V, as in the forward pass):
//       dQ_i = tril(G_i V_i^T) K_i + G_i S_{i-1}^T
//   reverse sweep  (running state T = sum over later chunks of Q^T G):
//       dK_i = tril(G_i V_i^T)^T Q_i + V_i T_i^T,     dV_i = tril(Q_i K_i^T)^T G_i + K_i T_i
// One CTA per (batch, head) does both sweeps; G is parked in the caller's workspace between them.
// The forward sweep recomputes r_t (nothing is saved by the forward pass).  Everything fp32 FFMA.
#include "common.cuh"

namespace chela {
namespace {

constexpr int kThreads = 256;

template <int D, int C>
struct BwdSmem {
    static constexpr int SS = D + 1;   // row stride of the running state: transposed reads stay spread over banks
    static constexpr int floats = 4 * C * D + D * SS + 2 * C * C;
};

// acc[r][s] += sum_{x < X} a(r, x) * b(x, s)
template <typename FA, typename FB>
__device__ __forceinline__ void mac_tile(float (&acc)[4][4], int X, FA a, FB b)
{
    for (int x = 0; x < X; ++x) {
        float av[4], bv[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) av[r] = a(r, x);
#pragma unroll
        for (int s = 0; s < 4; ++s) bv[s] = b(x, s);
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int s = 0; s < 4; ++s) acc[r][s] = fmaf(av[r], bv[s], acc[r][s]);
    }
}

template <int D, int C, typename TIn>
__global__ void __launch_bounds__(kThreads)
linattn_bwd_simt_kernel(const TIn *__restrict__ q, const TIn *__restrict__ k, const TIn *__restrict__ v,
                        const TIn *__restrict__ d_o, float *__restrict__ dq, float *__restrict__ dk, float *__restrict__ dv,
                        float *__restrict__ gbuf, int H, int L, float scale, int norm, float eps)
{
    extern __shared__ __align__(16) float smem[];
    constexpr int SS = BwdSmem<D, C>::SS;
    float *sQ = smem, *sK = sQ + C * D, *sV = sK + C * D, *sG = sV + C * D;   // [C][D] each
    float *sS = sG + C * D;                                                  // [D][SS] running state (S, then T)
    float *sP = sS + D * SS, *sA = sP + C * C;                               // [C][C] each
    const int tid = threadIdx.x;
    const int b = blockIdx.x / H, h = blockIdx.x % H;
    const size_t row_stride = (size_t)H * D;
    const size_t base = ((size_t)b * L * H + h) * D;
    const int nchunks = (L + C - 1) / C;

    auto load_tile = [&](float *dst, const auto *src, int t0, int n) {
        for (int idx = tid; idx < C * D / 4; idx += kThreads) {
            const int r = idx / (D / 4), c4 = (idx % (D / 4)) * 4;
            float4 f = make_float4(0.f, 0.f, 0.f, 0.f);
            if (r < n) f = load4(src + base + (size_t)(t0 + r) * row_stride + c4);
            store4(dst + r * D + c4, f);
        }
    };
    // tril(X Y^T) for [C][D] tiles X, Y -> out[C][C] (row a, column c, kept where c <= a)
    auto tril_xyT = [&](float *out, const float *X, const float *Y) {
        for (int tile = tid; tile < (C / 4) * (C / 4); tile += kThreads) {
            const int a0 = (tile / (C / 4)) * 4, c0 = (tile % (C / 4)) * 4;
            float acc[4][4] = {};
            if (c0 <= a0 + 3)
                mac_tile(acc, D, [&](int r, int x) { return X[(a0 + r) * D + x]; }, [&](int x, int s) { return Y[(c0 + s) * D + x]; });
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int s = 0; s < 4; ++s) out[(a0 + r) * C + c0 + s] = (c0 + s <= a0 + r) ? acc[r][s] : 0.f;
        }
    };
    auto zero_state = [&]() { for (int i = tid; i < D * SS; i += kThreads) sS[i] = 0.f; };
    // state[i][j] += sum_c X[c][i] * Y[c][j]
    auto update_state = [&](const float *X, const float *Y, int n) {
        for (int tile = tid; tile < (D / 4) * (D / 4); tile += kThreads) {
            const int i0 = (tile / (D / 4)) * 4, j0 = (tile % (D / 4)) * 4;
            float acc[4][4] = {};
            mac_tile(acc, n, [&](int r, int x) { return X[x * D + i0 + r]; }, [&](int x, int s) { return Y[x * D + j0 + s]; });
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int s = 0; s < 4; ++s) sS[(i0 + r) * SS + j0 + s] += acc[r][s];
        }
    };

    // ================================================= forward sweep: G, dQ ===============================
    zero_state();
    for (int ci = 0; ci < nchunks; ++ci) {
        const int t0 = ci * C, n = min(C, L - t0);
        load_tile(sQ, q, t0, n);
        load_tile(sK, k, t0, n);
        load_tile(sV, v, t0, n);
        load_tile(sG, d_o, t0, n);
        __syncthreads();
        tril_xyT(sP, sQ, sK);
        __syncthreads();
        // R = scale (Q S + P V); G = scale * normaliser-backward(dO, R); overwrites sG, parks G in gbuf
        for (int tile = tid; tile < (C / 4) * (D / 4); tile += kThreads) {
            const int a0 = (tile / (D / 4)) * 4, j0 = (tile % (D / 4)) * 4;
            float acc[4][4] = {};
            mac_tile(acc, D, [&](int r, int x) { return sQ[(a0 + r) * D + x]; }, [&](int x, int s) { return sS[x * SS + j0 + s]; });
            mac_tile(acc, min(a0 + 4, C), [&](int r, int x) { return sP[(a0 + r) * C + x]; }, [&](int x, int s) { return sV[x * D + j0 + s]; });
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                float g[4];
                if (norm) {
                    float ss = 0.f;
#pragma unroll
                    for (int s = 0; s < 4; ++s) {
                        acc[r][s] *= scale;
                        ss = fmaf(acc[r][s], acc[r][s], ss);
                    }
#pragma unroll
                    for (int m = D / 8; m >= 1; m >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, m, D / 4);
                    const float inv = rsqrtf(ss * (1.0f / D) + eps);
                    float od = 0.f;
#pragma unroll
                    for (int s = 0; s < 4; ++s) od = fmaf(acc[r][s] * inv, sG[(a0 + r) * D + j0 + s], od);
#pragma unroll
                    for (int m = D / 8; m >= 1; m >>= 1) od += __shfl_xor_sync(0xffffffffu, od, m, D / 4);
#pragma unroll
                    for (int s = 0; s < 4; ++s)
                        g[s] = scale * (sG[(a0 + r) * D + j0 + s] - acc[r][s] * inv * od * (1.0f / D)) * inv;
                } else {
#pragma unroll
                    for (int s = 0; s < 4; ++s) g[s] = scale * sG[(a0 + r) * D + j0 + s];
                }
                // every lane of the row has read its dO values above; the row's lanes write disjoint columns
                store4(sG + (a0 + r) * D + j0, make_float4(g[0], g[1], g[2], g[3]));
                if (a0 + r < n) store4(gbuf + base + (size_t)(t0 + a0 + r) * row_stride + j0, make_float4(g[0], g[1], g[2], g[3]));
            }
        }
        __syncthreads();
        tril_xyT(sA, sG, sV);
        __syncthreads();
        // dQ = A K + G S^T
        for (int tile = tid; tile < (C / 4) * (D / 4); tile += kThreads) {
            const int a0 = (tile / (D / 4)) * 4, i0 = (tile % (D / 4)) * 4;
            float acc[4][4] = {};
            mac_tile(acc, min(a0 + 4, C), [&](int r, int x) { return sA[(a0 + r) * C + x]; }, [&](int x, int s) { return sK[x * D + i0 + s]; });
            mac_tile(acc, D, [&](int r, int x) { return sG[(a0 + r) * D + x]; }, [&](int x, int s) { return sS[(i0 + s) * SS + x]; });
#pragma unroll
            for (int r = 0; r < 4; ++r)
                if (a0 + r < n) store4(dq + base + (size_t)(t0 + a0 + r) * row_stride + i0, make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]));
        }
        __syncthreads();
        update_state(sK, sV, n);
        __syncthreads();
    }

    // ================================================= reverse sweep: dK, dV ==============================
    zero_state();
    for (int ci = nchunks - 1; ci >= 0; --ci) {
        const int t0 = ci * C, n = min(C, L - t0);
        load_tile(sQ, q, t0, n);
        load_tile(sK, k, t0, n);
        load_tile(sV, v, t0, n);
        load_tile(sG, gbuf, t0, n);
        __syncthreads();
        tril_xyT(sP, sQ, sK);
        tril_xyT(sA, sG, sV);
        __syncthreads();
        for (int tile = tid; tile < (C / 4) * (D / 4); tile += kThreads) {
            const int c0 = (tile / (D / 4)) * 4, x0 = (tile % (D / 4)) * 4;
            // dK[c][i] = sum_{a >= c} A[a][c] Q[a][i] + sum_j V[c][j] T[i][j]
            float acc[4][4] = {};
            for (int a = c0; a < C; ++a) {
                float av[4], bv[4];
#pragma unroll
                for (int r = 0; r < 4; ++r) av[r] = sA[a * C + c0 + r];
#pragma unroll
                for (int s = 0; s < 4; ++s) bv[s] = sQ[a * D + x0 + s];
#pragma unroll
                for (int r = 0; r < 4; ++r)
#pragma unroll
                    for (int s = 0; s < 4; ++s) acc[r][s] = fmaf(av[r], bv[s], acc[r][s]);
            }
            mac_tile(acc, D, [&](int r, int x) { return sV[(c0 + r) * D + x]; }, [&](int x, int s) { return sS[(x0 + s) * SS + x]; });
#pragma unroll
            for (int r = 0; r < 4; ++r)
                if (c0 + r < n) store4(dk + base + (size_t)(t0 + c0 + r) * row_stride + x0, make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]));
            // dV[c][j] = sum_{a >= c} P[a][c] G[a][j] + sum_i K[c][i] T[i][j]
            float acc2[4][4] = {};
            for (int a = c0; a < C; ++a) {
                float av[4], bv[4];
#pragma unroll
                for (int r = 0; r < 4; ++r) av[r] = sP[a * C + c0 + r];
#pragma unroll
                for (int s = 0; s < 4; ++s) bv[s] = sG[a * D + x0 + s];
#pragma unroll
                for (int r = 0; r < 4; ++r)
#pragma unroll
                    for (int s = 0; s < 4; ++s) acc2[r][s] = fmaf(av[r], bv[s], acc2[r][s]);
            }
            mac_tile(acc2, D, [&](int r, int x) { return sK[(c0 + r) * D + x]; }, [&](int x, int s) { return sS[x * SS + x0 + s]; });
#pragma unroll
            for (int r = 0; r < 4; ++r)
                if (c0 + r < n) store4(dv + base + (size_t)(t0 + c0 + r) * row_stride + x0, make_float4(acc2[r][0], acc2[r][1], acc2[r][2], acc2[r][3]));
        }
        __syncthreads();
        update_state(sQ, sG, n);
        __syncthreads();
    }
}

template <int D, int C, typename TIn>
chela_status_t launch_t(const void *q, const void *k, const void *v, const void *d_o, float *dq, float *dk, float *dv,
                        float *gbuf, int B, int H, int L, int norm, float eps, float scale, cudaStream_t stream)
{
    auto kern = linattn_bwd_simt_kernel<D, C, TIn>;
    const size_t smem = sizeof(float) * BwdSmem<D, C>::floats;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return CHELA_ERR_CUDA;
    kern<<<B * H, kThreads, smem, stream>>>((const TIn *)q, (const TIn *)k, (const TIn *)v, (const TIn *)d_o, dq, dk, dv, gbuf, H, L,
                                           scale, norm, eps);
    return last_launch_status();
}

}  // namespace

size_t linattn_bwd_workspace_bytes(int B, int H, int L, int d) { return (size_t)B * L * H * d * sizeof(float); }

// In the rows of A and P beyond n the tiles are zero (loads zero-fill), so ragged tails need no special case.
chela_status_t launch_linattn_bwd_simt(const void *q, const void *k, const void *v, const void *d_o, float *dq, float *dk,
                                       float *dv, int B, int H, int L, int d, chela_dtype_t in_dtype, int norm, float eps,
                                       float scale, void *workspace, cudaStream_t stream)
{
    float *gbuf = (float *)workspace;
    if (d == 64) {
        if (in_dtype == CHELA_BF16) return launch_t<64, 64, __nv_bfloat16>(q, k, v, d_o, dq, dk, dv, gbuf, B, H, L, norm, eps, scale, stream);
        return launch_t<64, 64, float>(q, k, v, d_o, dq, dk, dv, gbuf, B, H, L, norm, eps, scale, stream);
    }
    if (d == 128) {
        if (in_dtype == CHELA_BF16) return launch_t<128, 32, __nv_bfloat16>(q, k, v, d_o, dq, dk, dv, gbuf, B, H, L, norm, eps, scale, stream);
        return launch_t<128, 32, float>(q, k, v, d_o, dq, dk, dv, gbuf, B, H, L, norm, eps, scale, stream);
    }
    return CHELA_ERR_UNSUPPORTED;
}

}  // namespace chela
