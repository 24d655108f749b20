// Chunked causal linear attention, fp32 SIMT kernel (Sec. 4.1 tiling; Eq. 2 with causal mask).
//
// One CTA per (batch, head).  Per chunk of C tokens it holds Q_i, K_i^T, V_i, the masked
// score tile P_i = tril(Q_i K_i^T) and the running state S = sum K^T V in shared memory, all fp32,
// and evaluates O_i = scale * (Q_i S_{i-1} + P_i V_i), the row normaliser, then S += K_i^T V_i.
// It serves the fp32 configuration (FFMA keeps the 1e-4 bound that single-pass TF32 would not)
// and is the in-library second opinion for the tensor-core kernel.
#include "common.cuh"

namespace chela {
namespace {

constexpr int kThreads = 256;

template <int D, int C>
struct SimtSmem {
    static constexpr int KS = C + 4;  // row stride of K^T, keeps float4 alignment
    static constexpr int floats = C * D + D * KS + C * D + D * D + C * C;
};

template <int D, int C, typename TIn, typename TOut>
__global__ void __launch_bounds__(kThreads)
linattn_simt_kernel(const TIn *__restrict__ q, const TIn *__restrict__ k, const TIn *__restrict__ v,
                    TOut *__restrict__ o, int H, int L, float scale, int norm, float eps,
                    const float *__restrict__ state_in, float *__restrict__ state_out)
{
    extern __shared__ __align__(16) float smem[];
    constexpr int KS = SimtSmem<D, C>::KS;
    float *sQ = smem;            // [C][D]
    float *sKt = sQ + C * D;     // [D][KS]   K transposed
    float *sV = sKt + D * KS;    // [C][D]
    float *sS = sV + C * D;      // [D][D]    running state, rows d_k, cols d_v
    float *sP = sS + D * D;      // [C][C]    masked scores

    const int tid = threadIdx.x;
    const int b = blockIdx.x / H, h = blockIdx.x % H;
    const size_t row_stride = (size_t)H * D;
    const size_t base = ((size_t)b * L * H + h) * D;

    // running state: zero, or the caller's initial state [B*H][D][D]
    for (int i = tid; i < D * D; i += kThreads) sS[i] = state_in ? state_in[(size_t)blockIdx.x * D * D + i] : 0.f;

    for (int t0 = 0; t0 < L; t0 += C) {
        const int n = min(C, L - t0);
        // ---- load chunk (rows >= n are zero) -------------------------------------------------
        for (int idx = tid; idx < C * D / 4; idx += kThreads) {
            const int r = idx / (D / 4), c4 = (idx % (D / 4)) * 4;
            float4 fq = make_float4(0.f, 0.f, 0.f, 0.f), fk = fq, fv = fq;
            if (r < n) {
                const size_t g = base + (size_t)(t0 + r) * row_stride + c4;
                fq = load4(q + g);
                fk = load4(k + g);
                fv = load4(v + g);
            }
            store4(sQ + r * D + c4, fq);
            store4(sV + r * D + c4, fv);
            sKt[(c4 + 0) * KS + r] = fk.x;
            sKt[(c4 + 1) * KS + r] = fk.y;
            sKt[(c4 + 2) * KS + r] = fk.z;
            sKt[(c4 + 3) * KS + r] = fk.w;
        }
        __syncthreads();
        // ---- P = tril(Q K^T) -----------------------------------------------------------------
        for (int tile = tid; tile < (C / 4) * (C / 4); tile += kThreads) {
            const int a0 = (tile / (C / 4)) * 4, c0 = (tile % (C / 4)) * 4;
            float acc[4][4] = {};
            if (c0 <= a0 + 3) {
                for (int i = 0; i < D; ++i) {
                    const float4 kk = load4(sKt + i * KS + c0);
                    const float kv[4] = {kk.x, kk.y, kk.z, kk.w};
#pragma unroll
                    for (int r = 0; r < 4; ++r) {
                        const float qv = sQ[(a0 + r) * D + i];
#pragma unroll
                        for (int s = 0; s < 4; ++s) acc[r][s] = fmaf(qv, kv[s], acc[r][s]);
                    }
                }
            }
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int s = 0; s < 4; ++s) sP[(a0 + r) * C + c0 + s] = (c0 + s <= a0 + r) ? acc[r][s] : 0.f;
        }
        __syncthreads();
        // ---- O = scale * (Q S + P V), normaliser, store ----------------------------------------
        for (int tile = tid; tile < (C / 4) * (D / 4); tile += kThreads) {
            const int a0 = (tile / (D / 4)) * 4, j0 = (tile % (D / 4)) * 4;
            float acc[4][4] = {};
            for (int i = 0; i < D; ++i) {
                const float4 sv = load4(sS + i * D + j0);
                const float s4[4] = {sv.x, sv.y, sv.z, sv.w};
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const float qv = sQ[(a0 + r) * D + i];
#pragma unroll
                    for (int s = 0; s < 4; ++s) acc[r][s] = fmaf(qv, s4[s], acc[r][s]);
                }
            }
            const int cend = min(a0 + 4, C);
            for (int c = 0; c < cend; ++c) {
                const float4 vv = load4(sV + c * D + j0);
                const float v4[4] = {vv.x, vv.y, vv.z, vv.w};
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const float pv = sP[(a0 + r) * C + c];
#pragma unroll
                    for (int s = 0; s < 4; ++s) acc[r][s] = fmaf(pv, v4[s], acc[r][s]);
                }
            }
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                float ss = 0.f;
#pragma unroll
                for (int s = 0; s < 4; ++s) {
                    acc[r][s] *= scale;
                    ss = fmaf(acc[r][s], acc[r][s], ss);
                }
                // the D/4 threads that share output row a0+r are consecutive lanes
#pragma unroll
                for (int m = D / 8; m >= 1; m >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, m, D / 4);
                const float inv = norm ? rsqrtf(ss * (1.0f / D) + eps) : 1.0f;
                if (a0 + r < n) {
                    const size_t g = base + (size_t)(t0 + a0 + r) * row_stride + j0;
                    store4(o + g, make_float4(acc[r][0] * inv, acc[r][1] * inv, acc[r][2] * inv, acc[r][3] * inv));
                }
            }
        }
        __syncthreads();
        // ---- S += K^T V ------------------------------------------------------------------------
        for (int tile = tid; tile < (D / 4) * (D / 4); tile += kThreads) {
            const int i0 = (tile / (D / 4)) * 4, j0 = (tile % (D / 4)) * 4;
            float acc[4][4] = {};
            for (int c = 0; c < n; ++c) {
                const float4 vv = load4(sV + c * D + j0);
                const float v4[4] = {vv.x, vv.y, vv.z, vv.w};
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const float kv = sKt[(i0 + r) * KS + c];
#pragma unroll
                    for (int s = 0; s < 4; ++s) acc[r][s] = fmaf(kv, v4[s], acc[r][s]);
                }
            }
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                float4 cur = load4(sS + (i0 + r) * D + j0);
                cur.x += acc[r][0]; cur.y += acc[r][1]; cur.z += acc[r][2]; cur.w += acc[r][3];
                store4(sS + (i0 + r) * D + j0, cur);
            }
        }
        __syncthreads();
    }
    if (state_out)
        for (int i = tid; i < D * D; i += kThreads) state_out[(size_t)blockIdx.x * D * D + i] = sS[i];
}

template <int D, int C, typename TIn, typename TOut>
chela_status_t launch_t(const void *q, const void *k, const void *v, void *o, int B, int H, int L,
                        int norm, float eps, float scale, cudaStream_t stream, const float *state_in, float *state_out)
{
    auto kern = linattn_simt_kernel<D, C, TIn, TOut>;
    const size_t smem = sizeof(float) * SimtSmem<D, C>::floats;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return CHELA_ERR_CUDA;
    kern<<<B * H, kThreads, smem, stream>>>((const TIn *)q, (const TIn *)k, (const TIn *)v, (TOut *)o, H, L,
                                           scale, norm, eps, state_in, state_out);
    return last_launch_status();
}

template <int D, int C>
chela_status_t launch_d(const void *q, const void *k, const void *v, void *o, int B, int H, int L,
                        chela_dtype_t in_dtype, chela_dtype_t out_dtype, int norm, float eps, float scale,
                        cudaStream_t stream, const float *state_in, float *state_out)
{
    if (in_dtype == CHELA_F32 && out_dtype == CHELA_F32)
        return launch_t<D, C, float, float>(q, k, v, o, B, H, L, norm, eps, scale, stream, state_in, state_out);
    if (in_dtype == CHELA_BF16 && out_dtype == CHELA_F32)
        return launch_t<D, C, __nv_bfloat16, float>(q, k, v, o, B, H, L, norm, eps, scale, stream, state_in, state_out);
    if (in_dtype == CHELA_BF16 && out_dtype == CHELA_BF16)
        return launch_t<D, C, __nv_bfloat16, __nv_bfloat16>(q, k, v, o, B, H, L, norm, eps, scale, stream, state_in, state_out);
    return launch_t<D, C, float, __nv_bfloat16>(q, k, v, o, B, H, L, norm, eps, scale, stream, state_in, state_out);
}

// ------------------------------------------------------------------------------- decode step
//
// One token per sequence with the state carried in place (recurrent form of Eq. 2):
//   S <- S + k v^T,   r = scale * S^T q,   o = Norm(r).
// One CTA of 256 threads per (batch, head).  The state is read and written exactly once (float4): the step is
// bound by those 2 * d * d * 4 bytes.  Thread t owns the four columns 4 * (t % (D/4)) of the rows
// t / (D/4) + j * (1024 / D); column sums are finished through shared memory.
template <int D, typename TIn, typename TOut>
__global__ void __launch_bounds__(256)
linattn_step_kernel(const TIn *__restrict__ q, const TIn *__restrict__ k, const TIn *__restrict__ v, TOut *__restrict__ o,
                    float *__restrict__ state, float scale, int norm, float eps)
{
    constexpr int CG = D / 4, RG = 256 / CG;   // column groups, row groups
    __shared__ float sq[D], sk[D];
    __shared__ float4 part[RG][CG];
    __shared__ float sr[D];
    const int tid = threadIdx.x, cg = tid % CG, rg = tid / CG;
    const size_t bh = blockIdx.x;
    if (tid < D) {
        sq[tid] = load1(q + bh * D + tid);
        sk[tid] = load1(k + bh * D + tid);
    }
    const float4 vv = load4(v + bh * D + 4 * cg);
    __syncthreads();
    float4 *S = reinterpret_cast<float4 *>(state + bh * D * D);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
    for (int i = rg; i < D; i += RG) {
        float4 sv = S[i * CG + cg];
        const float ki = sk[i], qi = sq[i];
        sv.x = fmaf(ki, vv.x, sv.x); sv.y = fmaf(ki, vv.y, sv.y); sv.z = fmaf(ki, vv.z, sv.z); sv.w = fmaf(ki, vv.w, sv.w);
        S[i * CG + cg] = sv;
        acc.x = fmaf(qi, sv.x, acc.x); acc.y = fmaf(qi, sv.y, acc.y); acc.z = fmaf(qi, sv.z, acc.z); acc.w = fmaf(qi, sv.w, acc.w);
    }
    part[rg][cg] = acc;
    __syncthreads();
    if (tid < CG) {
        float4 r = part[0][tid];
        for (int g = 1; g < RG; ++g) {
            const float4 p = part[g][tid];
            r.x += p.x; r.y += p.y; r.z += p.z; r.w += p.w;
        }
        r.x *= scale; r.y *= scale; r.z *= scale; r.w *= scale;
        *reinterpret_cast<float4 *>(sr + 4 * tid) = r;
    }
    __syncthreads();
    if (tid < 32) {
        float ss = 0.f;
        for (int j = tid; j < D; j += 32) ss = fmaf(sr[j], sr[j], ss);
#pragma unroll
        for (int m = 16; m >= 1; m >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, m);
        const float inv = norm ? rsqrtf(ss * (1.0f / D) + eps) : 1.0f;
        for (int j = tid; j < D; j += 32) store1(o + bh * D + j, sr[j] * inv);
    }
}

template <int D>
chela_status_t launch_step_d(const void *q, const void *k, const void *v, void *o, float *state, int B, int H,
                             chela_dtype_t in_dtype, chela_dtype_t out_dtype, int norm, float eps, float scale, cudaStream_t stream)
{
    const int grid = B * H;
    if (in_dtype == CHELA_F32 && out_dtype == CHELA_F32)
        linattn_step_kernel<D, float, float><<<grid, 256, 0, stream>>>((const float *)q, (const float *)k, (const float *)v, (float *)o, state, scale, norm, eps);
    else if (in_dtype == CHELA_F32)
        linattn_step_kernel<D, float, __nv_bfloat16><<<grid, 256, 0, stream>>>((const float *)q, (const float *)k, (const float *)v, (__nv_bfloat16 *)o, state, scale, norm, eps);
    else if (out_dtype == CHELA_F32)
        linattn_step_kernel<D, __nv_bfloat16, float><<<grid, 256, 0, stream>>>((const __nv_bfloat16 *)q, (const __nv_bfloat16 *)k, (const __nv_bfloat16 *)v, (float *)o, state, scale, norm, eps);
    else
        linattn_step_kernel<D, __nv_bfloat16, __nv_bfloat16><<<grid, 256, 0, stream>>>((const __nv_bfloat16 *)q, (const __nv_bfloat16 *)k, (const __nv_bfloat16 *)v, (__nv_bfloat16 *)o, state, scale, norm, eps);
    return last_launch_status();
}

}  // namespace

chela_status_t launch_linattn_step(const void *q, const void *k, const void *v, void *o, float *state, int B, int H, int d,
                                   chela_dtype_t in_dtype, chela_dtype_t out_dtype, int norm, float eps, float scale,
                                   cudaStream_t stream)
{
    if (d == 64) return launch_step_d<64>(q, k, v, o, state, B, H, in_dtype, out_dtype, norm, eps, scale, stream);
    if (d == 128) return launch_step_d<128>(q, k, v, o, state, B, H, in_dtype, out_dtype, norm, eps, scale, stream);
    return CHELA_ERR_UNSUPPORTED;
}

// The result does not depend on the chunk size; with d = 128 the shared-memory budget holds
// 64-token chunks only, so chunk = 128 is evaluated as two 64-token chunks there.
chela_status_t launch_linattn_simt(const void *q, const void *k, const void *v, void *o, int B, int H,
                                   int L, int d, int chunk, chela_dtype_t in_dtype,
                                   chela_dtype_t out_dtype, int norm, float eps, float scale,
                                   cudaStream_t stream, const float *state_in, float *state_out)
{
    if (d == 64 && chunk == 64) return launch_d<64, 64>(q, k, v, o, B, H, L, in_dtype, out_dtype, norm, eps, scale, stream, state_in, state_out);
    if (d == 64 && chunk == 128) return launch_d<64, 128>(q, k, v, o, B, H, L, in_dtype, out_dtype, norm, eps, scale, stream, state_in, state_out);
    if (d == 128) return launch_d<128, 64>(q, k, v, o, B, H, L, in_dtype, out_dtype, norm, eps, scale, stream, state_in, state_out);
    return CHELA_ERR_UNSUPPORTED;
}

}  // namespace chela
