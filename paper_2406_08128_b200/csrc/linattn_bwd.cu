// Backward of chunked causal linear attention on the tensor cores (bf16 inputs, d = 64), built from the
// forward kernel.  With G_t = scale * dLoss/dr_t (the output gradient pulled back through the normaliser),
// the three gradients are themselves linear attentions (Eq. 2 with the roles of the operands exchanged):
//   dQ = causal(q <- G, k <- V, v <- K)            dq_t = sum_{s<=t} <g_t,v_s> k_s
//   dK = anti-causal(q <- V, k <- G, v <- Q)       dk_s = sum_{t>=s} <v_s,g_t> q_t
//   dV = anti-causal(q <- K, k <- Q, v <- G)       dv_s = sum_{t>=s} <k_s,q_t> g_t
// so the pass is: the forward kernel without normaliser (recomputes r; nothing is saved by the forward pass),
// one elementwise kernel (r, d_o -> G), and three more launches of the forward kernel, two of them in its
// mirrored (anti-causal) mode.
// With the normaliser G is a bf16 pair (hi + lo): g_t is orthogonal to r_t up to eps / n_t^2, so dq, dk are
// residuals of a cancellation wherever n_t is small, and a G rounded to 8 bits loses them (measured 0.04-0.35
// of RMS).  The three launches then run the pair kernel with one real pair operand; the other two are single
// bf16 tensors whose absent low planes the copy engine zero-fills.  Without the normaliser G = scale * d_o is
// rounded to bf16 like every other operand and the single-bf16 kernel is used.
#include "common.cuh"

namespace chela {
namespace {

// one warp per (token, head) row of 64 values: G = scale * (d_o - o <o, d_o> / 64) / n, o = r / n,
// n = sqrt(mean r^2 + eps); without the normaliser G = scale * d_o.
__global__ void bwd_prep_kernel(const float *__restrict__ r, const __nv_bfloat16 *__restrict__ d_o,
                                __nv_bfloat16 *__restrict__ g, size_t rows, float scale, int norm, float eps)
{
    // with the normaliser g is written as a pair: low plane rows * 64 elements after the high plane
    const int lane = threadIdx.x & 31;
    const size_t warp = (blockIdx.x * (size_t)blockDim.x + threadIdx.x) >> 5, nwarps = ((size_t)gridDim.x * blockDim.x) >> 5;
    for (size_t row = warp; row < rows; row += nwarps) {
        const float2 dv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(d_o + row * 64 + 2 * lane));
        float2 out;
        if (norm) {
            const float2 rv = *reinterpret_cast<const float2 *>(r + row * 64 + 2 * lane);
            float ss = rv.x * rv.x + rv.y * rv.y;
#pragma unroll
            for (int m = 16; m >= 1; m >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, m);
            const float inv = rsqrtf(ss * (1.0f / 64) + eps);
            const float ox = rv.x * inv, oy = rv.y * inv;
            float od = ox * dv.x + oy * dv.y;
#pragma unroll
            for (int m = 16; m >= 1; m >>= 1) od += __shfl_xor_sync(0xffffffffu, od, m);
            od *= 1.0f / 64;
            out = make_float2(scale * (dv.x - ox * od) * inv, scale * (dv.y - oy * od) * inv);
        } else {
            out = make_float2(scale * dv.x, scale * dv.y);
        }
        const __nv_bfloat162 hi = __floats2bfloat162_rn(out.x, out.y);
        *reinterpret_cast<__nv_bfloat162 *>(g + row * 64 + 2 * lane) = hi;
        if (norm) {
            const float2 hf = __bfloat1622float2(hi);
            *reinterpret_cast<__nv_bfloat162 *>(g + (rows + row) * 64 + 2 * lane) = __floats2bfloat162_rn(out.x - hf.x, out.y - hf.y);
        }
    }
}

}  // namespace

bool linattn_bwd_sm100_supported(int d, chela_dtype_t in_dtype) { return d == 64 && in_dtype == CHELA_BF16; }

// attention workspace | r (fp32) | G (bf16 pair)
size_t linattn_bwd_sm100_workspace_bytes(int B, int H, int L)
{
    const size_t n = (size_t)B * L * H * 64;
    return align_up(linattn_sm100_workspace_bytes(B, H, L, 64, 64), 256) + n * sizeof(float) + 2 * n * sizeof(__nv_bfloat16);
}

chela_status_t launch_linattn_bwd_sm100(const void *q, const void *k, const void *v, const void *d_o, float *dq, float *dk,
                                        float *dv, int B, int H, int L, int norm, float eps, float scale, void *workspace,
                                        cudaStream_t stream)
{
    const size_t n = (size_t)B * L * H * 64, rows = (size_t)B * L * H;
    char *ws = (char *)workspace;
    void *attn_ws = ws;
    float *r = (float *)(ws + align_up(linattn_sm100_workspace_bytes(B, H, L, 64, 64), 256));
    __nv_bfloat16 *g = (__nv_bfloat16 *)(r + n);
    chela_status_t st = CHELA_OK;
    if (norm)   // r_t = scale * sum_{s<=t} <q_t,k_s> v_s
        st = launch_linattn_sm100(q, k, v, r, B, H, L, 64, 64, CHELA_BF16, CHELA_F32, 0, eps, scale, attn_ws, stream);
    if (st != CHELA_OK) return st;
    const int blocks = (int)((rows + 7) / 8 < (size_t)148 * 16 ? (rows + 7) / 8 : (size_t)148 * 16);
    bwd_prep_kernel<<<blocks, 256, 0, stream>>>(r, (const __nv_bfloat16 *)d_o, g, rows, scale, norm, eps);
    if (cudaGetLastError() != cudaSuccess) return CHELA_ERR_CUDA;
    const chela_dtype_t dt = norm ? CHELA_BF16_PAIR : CHELA_BF16;   // the pair is G, in a different role each time
    st = launch_linattn_sm100(g, v, k, dq, B, H, L, 64, 64, dt, CHELA_F32, 0, eps, 1.0f, attn_ws, stream, nullptr, nullptr, false, 1);
    if (st != CHELA_OK) return st;
    st = launch_linattn_sm100(v, g, q, dk, B, H, L, 64, 64, dt, CHELA_F32, 0, eps, 1.0f, attn_ws, stream, nullptr, nullptr, true, 2);
    if (st != CHELA_OK) return st;
    return launch_linattn_sm100(k, q, g, dv, B, H, L, 64, 64, dt, CHELA_F32, 0, eps, 1.0f, attn_ws, stream, nullptr, nullptr, true, 4);
}

}  // namespace chela
