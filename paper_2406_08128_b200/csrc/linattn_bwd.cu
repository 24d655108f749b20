// Backward of chunked causal linear attention on the tensor cores (bf16 inputs, d = 64 or 128), built from the
// forward kernel.  With G_t = scale * dLoss/dr_t (the output gradient pulled back through the normaliser),
// the three gradients are themselves linear attentions (Eq. 2 with the roles of the operands exchanged):
//   dQ = causal(q <- G, k <- V, v <- K)            dq_t = sum_{s<=t} <g_t,v_s> k_s
//   dK = anti-causal(q <- V, k <- G, v <- Q)       dk_s = sum_{t>=s} <v_s,g_t> q_t
//   dV = anti-causal(q <- K, k <- Q, v <- G)       dv_s = sum_{t>=s} <k_s,q_t> g_t
// so the pass is four launches of the forward kernel (nothing is saved by the forward pass): one that recomputes
// r and writes G from its epilogue (d = 64; for d = 128 the forward kernel writes r and an elementwise kernel
// makes G), and three that evaluate the gradients, two of them in the mirrored (anti-causal) mode.
// With the normaliser G is a bf16 pair (hi + lo): g_t is orthogonal to r_t up to eps / n_t^2, so dq, dk are
// residuals of a cancellation wherever n_t is small, and a G rounded to 8 bits loses them (measured 0.04-0.35
// of RMS); r itself, which the normaliser differentiates through, is recomputed with scores and state kept as
// pairs, and so are the scores of the gradient launches (single-bf16 scores there: 1-3e-2 of RMS).  Each
// gradient launch has one pair operand (G, in a different role each time) and runs the kernel variant that
// carries exactly that low plane.  Without the normaliser G = scale * d_o: the launches take d_o itself, the
// factor goes into their scale argument, and the plain bf16 kernel is used.
#include "common.cuh"

namespace chela {
namespace {

// one warp per (token, head) row of D values: G = scale * (d_o - o <o, d_o> / D) / n, o = r / n,
// n = sqrt(mean r^2 + eps); without the normaliser G = scale * d_o.
template <int D>
__global__ void bwd_prep_kernel(const float *__restrict__ r, const __nv_bfloat16 *__restrict__ d_o,
                                __nv_bfloat16 *__restrict__ g, size_t rows, float scale, int norm, float eps)
{
    // with the normaliser g is written as a pair: low plane rows * D elements after the high plane
    constexpr int V = D / 64;   // bf16x2 / float2 items per lane
    const int lane = threadIdx.x & 31;
    const size_t warp = (blockIdx.x * (size_t)blockDim.x + threadIdx.x) >> 5, nwarps = ((size_t)gridDim.x * blockDim.x) >> 5;
    for (size_t row = warp; row < rows; row += nwarps) {
        float2 dv[V], out[V];
#pragma unroll
        for (int i = 0; i < V; ++i)
            dv[i] = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(d_o + row * D + 2 * (lane + 32 * i)));
        if (norm) {
            float2 rv[V];
            float ss = 0.f;
#pragma unroll
            for (int i = 0; i < V; ++i) {
                rv[i] = *reinterpret_cast<const float2 *>(r + row * D + 2 * (lane + 32 * i));
                ss += rv[i].x * rv[i].x + rv[i].y * rv[i].y;
            }
#pragma unroll
            for (int m = 16; m >= 1; m >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, m);
            const float inv = rsqrtf(ss * (1.0f / D) + eps);
            float od = 0.f;
#pragma unroll
            for (int i = 0; i < V; ++i) od += rv[i].x * inv * dv[i].x + rv[i].y * inv * dv[i].y;
#pragma unroll
            for (int m = 16; m >= 1; m >>= 1) od += __shfl_xor_sync(0xffffffffu, od, m);
            od *= 1.0f / D;
#pragma unroll
            for (int i = 0; i < V; ++i)
                out[i] = make_float2(scale * (dv[i].x - rv[i].x * inv * od) * inv, scale * (dv[i].y - rv[i].y * inv * od) * inv);
        } else {
#pragma unroll
            for (int i = 0; i < V; ++i) out[i] = make_float2(scale * dv[i].x, scale * dv[i].y);
        }
#pragma unroll
        for (int i = 0; i < V; ++i) {
            const size_t at = row * D + 2 * (lane + 32 * i);
            const __nv_bfloat162 hi = __floats2bfloat162_rn(out[i].x, out[i].y);
            *reinterpret_cast<__nv_bfloat162 *>(g + at) = hi;
            if (norm) {
                const float2 hf = __bfloat1622float2(hi);
                *reinterpret_cast<__nv_bfloat162 *>(g + rows * D + at) = __floats2bfloat162_rn(out[i].x - hf.x, out[i].y - hf.y);
            }
        }
    }
}

}  // namespace

bool linattn_bwd_sm100_supported(int d, chela_dtype_t in_dtype) { return (d == 64 || d == 128) && in_dtype == CHELA_BF16; }

// attention workspace | r (fp32) | G (bf16 pair)
size_t linattn_bwd_sm100_workspace_bytes(int B, int H, int L, int d)
{
    const size_t n = (size_t)B * L * H * d;
    return align_up(linattn_sm100_workspace_bytes(B, H, L, d, 64), 256) + n * sizeof(float) + 2 * n * sizeof(__nv_bfloat16);
}

chela_status_t launch_linattn_bwd_sm100(const void *q, const void *k, const void *v, const void *d_o, float *dq, float *dk,
                                        float *dv, int B, int H, int L, int d, int norm, float eps, float scale,
                                        void *workspace, cudaStream_t stream)
{
    const size_t n = (size_t)B * L * H * d, rows = (size_t)B * L * H;
    char *ws = (char *)workspace;
    void *attn_ws = ws;
    float *r = (float *)(ws + align_up(linattn_sm100_workspace_bytes(B, H, L, d, 64), 256));
    __nv_bfloat16 *g = (__nv_bfloat16 *)(r + n);
    chela_status_t st = CHELA_OK;
    const void *gp = g;
    float gscale = 1.0f;
    // the launches share one status word: only the first of them clears it, so a timeout in any of them is still
    // there when the caller looks
    bool keep = false;
    if (!norm) {
        // G = scale * d_o: the gradient launches take d_o itself and the factor
        gp = d_o;
        gscale = scale;
    } else if (d == 64) {
        // one launch recomputes r (scores and state kept as bf16 pairs: the normaliser differentiates through r,
        // which therefore has to be good to fp32 rather than to bf16 scores) and writes G from its epilogue
        st = launch_linattn_sm100_grad(q, k, v, d_o, g, B, H, L, eps, scale, attn_ws, stream);
        if (st != CHELA_OK) return st;
        keep = true;
    } else {
        // d = 128: r from the pair kernel with every low input plane absent, then G by an elementwise kernel
        st = launch_linattn_sm100(q, k, v, r, B, H, L, d, 64, CHELA_BF16_PAIR, CHELA_F32, 0, eps, scale, attn_ws, stream,
                                  nullptr, nullptr, false, 0);
        if (st != CHELA_OK) return st;
        keep = true;
        const int blocks = (int)((rows + 7) / 8 < (size_t)148 * 16 ? (rows + 7) / 8 : (size_t)148 * 16);
        bwd_prep_kernel<128><<<blocks, 256, 0, stream>>>(r, (const __nv_bfloat16 *)d_o, g, rows, scale, norm, eps);
        if (cudaGetLastError() != cudaSuccess) return CHELA_ERR_CUDA;
    }
    const chela_dtype_t dt = norm ? CHELA_BF16_PAIR : CHELA_BF16;   // the pair is G, in a different role each time
    st = launch_linattn_sm100(gp, v, k, dq, B, H, L, d, 64, dt, CHELA_F32, 0, eps, gscale, attn_ws, stream, nullptr, nullptr, false, 1, keep);
    if (st != CHELA_OK) return st;
    st = launch_linattn_sm100(v, gp, q, dk, B, H, L, d, 64, dt, CHELA_F32, 0, eps, gscale, attn_ws, stream, nullptr, nullptr, true, 2, true);
    if (st != CHELA_OK) return st;
    return launch_linattn_sm100(k, q, gp, dv, B, H, L, d, 64, dt, CHELA_F32, 0, eps, gscale, attn_ws, stream, nullptr, nullptr, true, 4, true);
}

}  // namespace chela
