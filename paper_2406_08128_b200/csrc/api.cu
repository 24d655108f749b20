// C ABI entry points: argument validation, workspace carving and dispatch.  No kernel code here.
#include <cmath>

#include "common.cuh"

using namespace chela;

namespace {
constexpr int kLongconvMaxL = 262144;   // 16 blocks of the blocked long convolution

bool dtype_ok(chela_dtype_t t) { return t == CHELA_F32 || t == CHELA_BF16; }

struct MixerPlan {
    size_t off_conv, off_z, off_q, off_k, off_v, off_attn, off_ga, off_go, off_o, total;
    size_t conv_bytes, attn_bytes;
};
MixerPlan mixer_plan(int B, int L, int D, int H, int chunk, bool gated)
{
    MixerPlan p;
    const size_t act = align_up((size_t)B * L * D * sizeof(float), 256);
    p.conv_bytes = longconv_workspace_bytes(B, L, D);
    p.attn_bytes = chela_linattn_workspace_bytes(B, H, L, D / H, D / H, chunk);
    p.off_attn = 0;  // first, so that the asynchronous status word heads the mixer workspace too
    p.off_conv = align_up(p.attn_bytes, 256);
    p.off_z = p.off_conv + align_up(p.conv_bytes, 256);
    p.off_q = p.off_z + act;
    p.off_k = p.off_q + act;
    p.off_v = p.off_k + act;
    p.off_ga = p.off_v + act;                 // gated form only: G_a, G_o, un-gated attention output
    p.off_go = p.off_ga + (gated ? act : 0);
    p.off_o = p.off_go + (gated ? act : 0);
    p.total = p.off_o + (gated ? act : 0);
    return p;
}

// Room for a copy of the initial state of chela_linattn_carry_fwd, behind the kernels' own workspace: needed when
// state_in and state_out are the same buffer and a sequence may be shared between CTAs (fewer pairs than SMs).
size_t carry_staging_bytes(int B, int H, int d)
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        sms = 148;
    (void)cudaGetLastError();
    if ((long long)B * H >= sms) return 0;
    return 256 + (size_t)B * H * d * d * sizeof(float);
}

// what chela_debug_wait_control last set; process-wide, read by every tensor-core launch
long long g_wait_limit_cycles = 2000000000LL;   // about one second at B200 clocks
int g_skip_arrival = 0;

}  // namespace

namespace chela {
WaitCtl current_wait_ctl() { return WaitCtl{g_wait_limit_cycles, g_skip_arrival}; }
}  // namespace chela

extern "C" {

namespace {
__global__ void sm_clock_probe_kernel(long long *out, long long spin_cycles)
{
    unsigned long long g0, g1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g0));
    const long long c0 = clock64();
    long long c1 = c0;
    while (c1 - c0 < spin_cycles) c1 = clock64();   // bounded by spin_cycles
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g1));
    out[0] = c1 - c0;
    out[1] = (long long)(g1 - g0);
}
}  // namespace

chela_status_t chela_debug_sm_clock(void *out16, long long spin_cycles, cudaStream_t stream)
{
    if (!out16 || (reinterpret_cast<uintptr_t>(out16) & 7u)) return CHELA_ERR_INVALID_ARG;
    if (spin_cycles < 10000) spin_cycles = 10000;
    if (spin_cycles > 2000000) spin_cycles = 2000000;
    sm_clock_probe_kernel<<<1, 1, 0, stream>>>((long long *)out16, spin_cycles);
    return last_launch_status();
}

void chela_debug_wait_control(long long limit_cycles, int skip_arrival)
{
    g_wait_limit_cycles = limit_cycles > 0 ? limit_cycles : 2000000000LL;
    g_skip_arrival = skip_arrival;
}

const char *chela_status_string(chela_status_t status)
{
    switch (status) {
        case CHELA_OK: return "ok";
        case CHELA_ERR_INVALID_ARG: return "invalid argument";
        case CHELA_ERR_UNSUPPORTED: return "unsupported shape or dtype";
        case CHELA_ERR_WORKSPACE: return "workspace missing or too small";
        case CHELA_ERR_CUDA: return "CUDA call failed";
        case CHELA_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

int chela_version(void) { return 100; }

int chela_linattn_kernel_kind(int B, int H, int L, int d_k, int d_v, int chunk, chela_dtype_t in_dtype,
                              chela_dtype_t out_dtype)
{
    if (B < 1 || H < 1 || L < 1 || !(dtype_ok(in_dtype) || in_dtype == CHELA_BF16_PAIR) || !dtype_ok(out_dtype)) return 0;
    if (d_k != d_v || (d_k != 64 && d_k != 128) || (chunk != 64 && chunk != 128)) return 0;
    if (linattn_sm100_supported(B, H, L, d_k, chunk, in_dtype, out_dtype)) return 2;
    return in_dtype == CHELA_BF16_PAIR ? 0 : 1;
}

int chela_linattn_split_plan(int B, int H, int L, int d, chela_dtype_t in_dtype, int sms, int *groups, int *first_chunks,
                             int *other_chunks)
{
    if (B < 1 || H < 1 || L < 1 || (d != 64 && d != 128) || !groups || !first_chunks || !other_chunks) return 0;
    linattn_sm100_split(B, H, L, d, in_dtype == CHELA_BF16_PAIR, sms, groups, first_chunks, other_chunks);
    return 1;
}

chela_status_t chela_shortconv_fwd(const void *x, const float *w, const float *bias, void *y, int B, int L,
                                   int D, int width, int act, chela_dtype_t io_dtype, cudaStream_t stream)
{
    if (!x || !w || !y || x == y || B < 1 || L < 1 || D < 1 || !dtype_ok(io_dtype) || (act != 0 && act != 1))
        return CHELA_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(y)) return CHELA_ERR_INVALID_ARG;
    if (width < 1 || width > 16 || D % 8 != 0) return CHELA_ERR_UNSUPPORTED;
    return launch_shortconv(x, w, bias, y, B, L, D, width, act, io_dtype, stream);
}

int chela_second_short_width(int L)
{
    if (L < 1) return 1;
    const double w = 2.0 * log10((double)L) + 1.0;
    int odd = 2 * (int)floor(w / 2.0) + 1;   // odd integers around w: odd <= w < odd + 2 (or odd - 2 < w)
    if (w - odd > odd + 2 - w) odd += 2;
    if (odd - w > w - (odd - 2)) odd -= 2;
    return odd < 1 ? 1 : (odd > 15 ? 15 : odd);
}

chela_status_t chela_shortconv_reparam(const float *w1, int width1, const float *w2, int width2, float *merged, int D,
                                       cudaStream_t stream)
{
    if (!w1 || !w2 || !merged || D < 1 || width1 < 1 || width2 < 1) return CHELA_ERR_INVALID_ARG;
    if (width1 > 16 || width2 > 16) return CHELA_ERR_UNSUPPORTED;
    return launch_shortconv_reparam(w1, width1, w2, width2, merged, D, stream);
}

size_t chela_longconv_workspace_bytes(int B, int L, int D, chela_dtype_t, chela_dtype_t)
{
    if (B < 1 || L < 1 || D < 1) return 0;
    return longconv_workspace_bytes(B, L, D);
}

size_t chela_longconv_spectrum_bytes(int L, int D)
{
    if (L < 1 || L > kLongconvMaxL || D < 1 || D % 8 != 0) return 0;
    return longconv_spectrum_bytes(L, D);
}

chela_status_t chela_longconv_prepare(const float *k_long, int L, int D, void *spectrum, size_t spectrum_bytes, cudaStream_t stream)
{
    if (!k_long || !spectrum || L < 1 || D < 1 || !aligned16(spectrum)) return CHELA_ERR_INVALID_ARG;
    if (L > kLongconvMaxL || D % 8 != 0) return CHELA_ERR_UNSUPPORTED;
    if (spectrum_bytes < longconv_spectrum_bytes(L, D)) return CHELA_ERR_WORKSPACE;
    return launch_longconv_prepare(k_long, L, D, spectrum, stream);
}

chela_status_t chela_longconv_prepared_fwd(const void *x, const void *spectrum, const float *w_short, int short_width,
                                           void *z, int B, int L, int D, chela_dtype_t in_dtype, chela_dtype_t out_dtype,
                                           void *workspace, size_t workspace_bytes, cudaStream_t stream)
{
    if (!x || !spectrum || !z || B < 1 || L < 1 || D < 1 || !dtype_ok(in_dtype) || !dtype_ok(out_dtype))
        return CHELA_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(z) || !aligned16(workspace) || !aligned16(spectrum)) return CHELA_ERR_INVALID_ARG;
    if (L > kLongconvMaxL || D % 8 != 0) return CHELA_ERR_UNSUPPORTED;
    if (w_short && (short_width < 1 || short_width > 16)) return CHELA_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < longconv_workspace_bytes(B, L, D)) return CHELA_ERR_WORKSPACE;
    return launch_longconv(x, nullptr, w_short, short_width, z, B, L, D, in_dtype, out_dtype, workspace, stream, false, spectrum);
}

chela_status_t chela_longconv_fwd(const void *x, const float *k_long, const float *w_short, int short_width,
                                  void *z, int B, int L, int D, chela_dtype_t in_dtype,
                                  chela_dtype_t out_dtype, void *workspace, size_t workspace_bytes,
                                  cudaStream_t stream)
{
    if (!x || !k_long || !z || B < 1 || L < 1 || D < 1 || !dtype_ok(in_dtype) || !dtype_ok(out_dtype))
        return CHELA_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(z) || !aligned16(workspace)) return CHELA_ERR_INVALID_ARG;
    if (L > kLongconvMaxL || D % 8 != 0) return CHELA_ERR_UNSUPPORTED;
    if (w_short && (short_width < 1 || short_width > 16)) return CHELA_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < longconv_workspace_bytes(B, L, D)) return CHELA_ERR_WORKSPACE;
    return launch_longconv(x, k_long, w_short, short_width, z, B, L, D, in_dtype, out_dtype, workspace, stream);
}

size_t chela_linattn_workspace_bytes(int B, int H, int L, int d_k, int d_v, int chunk)
{
    if (B < 1 || H < 1 || L < 1 || d_k != d_v || (d_k != 64 && d_k != 128) || (chunk != 64 && chunk != 128))
        return 0;
    return linattn_sm100_workspace_bytes(B, H, L, d_k, chunk) + carry_staging_bytes(B, H, d_k);
}

chela_status_t chela_linattn_carry_fwd(const void *q, const void *k, const void *v, void *o, const float *state_in,
                                       float *state_out, int B, int H, int L, int d_k, int d_v, int chunk,
                                       chela_dtype_t in_dtype, chela_dtype_t out_dtype, chela_norm_t norm,
                                       float norm_eps, float scale, void *workspace, size_t workspace_bytes,
                                       cudaStream_t stream)
{
    if (!q || !k || !v || !o || B < 1 || H < 1 || L < 1 || d_k < 1 || d_v < 1 || chunk < 1 ||
        !(dtype_ok(in_dtype) || in_dtype == CHELA_BF16_PAIR) || !dtype_ok(out_dtype) ||
        (norm != CHELA_NORM_NONE && norm != CHELA_NORM_RMS) || !(norm_eps >= 0.f))
        return CHELA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(workspace) ||
        !aligned16(state_in) || !aligned16(state_out))
        return CHELA_ERR_INVALID_ARG;
    const int kind = chela_linattn_kernel_kind(B, H, L, d_k, d_v, chunk, in_dtype, out_dtype);
    if (kind == 0) return CHELA_ERR_UNSUPPORTED;
    if (kind == 2) {
        const size_t base = linattn_sm100_workspace_bytes(B, H, L, d_k, chunk), staging = carry_staging_bytes(B, H, d_k);
        if (!workspace || workspace_bytes < base + staging) return CHELA_ERR_WORKSPACE;
        if (state_in && state_in == state_out && staging) {
            // A sequence may be shared between several CTAs (few (batch, head) pairs): every one of them reads the initial
            // state when it starts, one writes the final state when it ends, and nothing orders the two across CTAs.  With
            // aliased pointers the initial state is therefore read from a copy taken on the stream first.
            float *copy = reinterpret_cast<float *>(static_cast<char *>(workspace) + align_up(base, 256));
            if (cudaMemcpyAsync(copy, state_in, (size_t)B * H * d_k * d_k * sizeof(float), cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
                return CHELA_ERR_CUDA;
            state_in = copy;
        }
        return launch_linattn_sm100(q, k, v, o, B, H, L, d_k, chunk, in_dtype, out_dtype, (int)norm, norm_eps,
                                    scale, workspace, stream, state_in, state_out);
    }
    return launch_linattn_simt(q, k, v, o, B, H, L, d_k, chunk, in_dtype, out_dtype, (int)norm, norm_eps, scale,
                               stream, state_in, state_out);
}

chela_status_t chela_linattn_fwd(const void *q, const void *k, const void *v, void *o, int B, int H, int L,
                                 int d_k, int d_v, int chunk, chela_dtype_t in_dtype,
                                 chela_dtype_t out_dtype, chela_norm_t norm, float norm_eps, float scale,
                                 void *workspace, size_t workspace_bytes, cudaStream_t stream)
{
    return chela_linattn_carry_fwd(q, k, v, o, nullptr, nullptr, B, H, L, d_k, d_v, chunk, in_dtype, out_dtype, norm,
                                   norm_eps, scale, workspace, workspace_bytes, stream);
}

chela_status_t chela_linattn_step(const void *q, const void *k, const void *v, void *o, float *state, int B, int H,
                                  int d_k, int d_v, chela_dtype_t in_dtype, chela_dtype_t out_dtype, chela_norm_t norm,
                                  float norm_eps, float scale, cudaStream_t stream)
{
    if (!q || !k || !v || !o || !state || B < 1 || H < 1 || d_k < 1 || d_v < 1 || !dtype_ok(in_dtype) || !dtype_ok(out_dtype) ||
        (norm != CHELA_NORM_NONE && norm != CHELA_NORM_RMS) || !(norm_eps >= 0.f))
        return CHELA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(state)) return CHELA_ERR_INVALID_ARG;
    if (d_k != d_v || (d_k != 64 && d_k != 128)) return CHELA_ERR_UNSUPPORTED;
    return launch_linattn_step(q, k, v, o, state, B, H, d_k, in_dtype, out_dtype, (int)norm, norm_eps, scale, stream);
}

size_t chela_linattn_bwd_workspace_bytes(int B, int H, int L, int d_k, int d_v)
{
    if (B < 1 || H < 1 || L < 1 || d_k != d_v || (d_k != 64 && d_k != 128)) return 0;
    const size_t simt = linattn_bwd_workspace_bytes(B, H, L, d_k);
    const size_t tensor = linattn_bwd_sm100_workspace_bytes(B, H, L, d_k);   // the query does not know the dtype
    return simt > tensor ? simt : tensor;
}

chela_status_t chela_linattn_bwd(const void *q, const void *k, const void *v, const void *d_o, float *dq, float *dk,
                                 float *dv, int B, int H, int L, int d_k, int d_v, chela_dtype_t in_dtype,
                                 chela_norm_t norm, float norm_eps, float scale, void *workspace, size_t workspace_bytes,
                                 cudaStream_t stream)
{
    if (!q || !k || !v || !d_o || !dq || !dk || !dv || B < 1 || H < 1 || L < 1 || !dtype_ok(in_dtype) ||
        (norm != CHELA_NORM_NONE && norm != CHELA_NORM_RMS) || !(norm_eps >= 0.f))
        return CHELA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(d_o) || !aligned16(dq) || !aligned16(dk) ||
        !aligned16(dv) || !aligned16(workspace))
        return CHELA_ERR_INVALID_ARG;
    if (d_k != d_v || (d_k != 64 && d_k != 128)) return CHELA_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < chela_linattn_bwd_workspace_bytes(B, H, L, d_k, d_v)) return CHELA_ERR_WORKSPACE;
    if (linattn_bwd_sm100_supported(d_k, in_dtype))
        return launch_linattn_bwd_sm100(q, k, v, d_o, dq, dk, dv, B, H, L, d_k, (int)norm, norm_eps, scale, workspace, stream);
    return launch_linattn_bwd_simt(q, k, v, d_o, dq, dk, dv, B, H, L, d_k, in_dtype, (int)norm, norm_eps, scale, workspace,
                                   stream);
}

size_t chela_dense_workspace_bytes(void) { return 256; }

chela_status_t chela_dense_fwd(const void *a, const void *w, const float *bias, void *y, int M, int K, int N, int act,
                               chela_dtype_t a_dtype, chela_dtype_t w_dtype, chela_dtype_t y_dtype, void *workspace,
                               size_t workspace_bytes, cudaStream_t stream)
{
    auto any_dtype = [](chela_dtype_t t) { return t == CHELA_F32 || t == CHELA_BF16 || t == CHELA_BF16_PAIR; };
    if (!a || !w || !y || M < 1 || K < 1 || N < 1 || (act < 0 || act > 2) || !any_dtype(a_dtype) || !dtype_ok(w_dtype) ||
        !any_dtype(y_dtype))
        return CHELA_ERR_INVALID_ARG;
    if (!aligned16(a) || !aligned16(w) || !aligned16(y) || !aligned16(workspace)) return CHELA_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < chela_dense_workspace_bytes()) return CHELA_ERR_WORKSPACE;
    if (cudaMemsetAsync(workspace, 0, 2 * sizeof(int), stream) != cudaSuccess) return CHELA_ERR_CUDA;
    if (gemm_sm100_supported((size_t)M, K, N, a_dtype, w_dtype, y_dtype))
        return launch_gemm_sm100(a, w, bias, y, (size_t)M, K, N, act, a_dtype, y_dtype, (int *)workspace, stream);
    if (a_dtype == CHELA_BF16_PAIR || y_dtype == CHELA_BF16_PAIR) return CHELA_ERR_UNSUPPORTED;
    return launch_gemm_simt(a, w, bias, y, (size_t)M, K, N, act, a_dtype, w_dtype, y_dtype, stream);
}

chela_status_t chela_async_status(const void *workspace, cudaStream_t stream)
{
    if (!workspace) return CHELA_ERR_INVALID_ARG;
    int word[2] = {0, 0};   // word 0: attention kernels (or the only kernel of the call); word 1: the mixer's GEMMs
    if (cudaMemcpyAsync(word, workspace, sizeof(word), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess)
        return CHELA_ERR_CUDA;
    if (word[0] == (int)CHELA_ERR_TIMEOUT || word[1] == (int)CHELA_ERR_TIMEOUT) return CHELA_ERR_TIMEOUT;
    if (word[0] == (int)CHELA_ERR_CUDA || word[1] == (int)CHELA_ERR_CUDA) return CHELA_ERR_CUDA;
    return CHELA_OK;
}

size_t chela_mixer_workspace_bytes(int B, int L, int D, int H, int chunk, chela_dtype_t)
{
    if (B < 1 || L < 1 || D < 1 || H < 1 || D % H != 0) return 0;
    return mixer_plan(B, L, D, H, chunk, false).total;
}

size_t chela_mixer_gated_workspace_bytes(int B, int L, int D, int H, int chunk, chela_dtype_t)
{
    if (B < 1 || L < 1 || D < 1 || H < 1 || D % H != 0) return 0;
    return mixer_plan(B, L, D, H, chunk, true).total;
}

}  // extern "C"

namespace {
chela_status_t mixer_impl(const void *x, const float *w_short, int short_width, const float *k_long, const void *spectrum, const void *w_q,
                          const void *w_k, const void *w_v, const float *b_q, const float *b_k, const float *b_v,
                          const void *w_a, const float *b_a, const void *w_o, const float *b_o, int qk_diag, int v_silu,
                          void *o, int B, int L, int D, int H, int chunk, chela_dtype_t in_dtype, chela_dtype_t out_dtype,
                          chela_norm_t norm, float norm_eps, void *workspace, size_t workspace_bytes, cudaStream_t stream)
{
    const bool gated = w_a != nullptr;
    if (gated && !w_o) return CHELA_ERR_INVALID_ARG;
    if (!x || !w_short || (!k_long && !spectrum) || !aligned16(spectrum) || !w_q || !w_k || !w_v || !o || B < 1 || L < 1 || D < 1 || H < 1 ||
        !dtype_ok(in_dtype) || !dtype_ok(out_dtype) || (norm != CHELA_NORM_NONE && norm != CHELA_NORM_RMS) ||
        !(norm_eps >= 0.f))
        return CHELA_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(o) || !aligned16(w_q) || !aligned16(w_k) || !aligned16(w_v) ||
        !aligned16(workspace) || !aligned16(w_a) || !aligned16(w_o))
        return CHELA_ERR_INVALID_ARG;
    if (D % H != 0) return CHELA_ERR_INVALID_ARG;
    const int d = D / H;
    if ((d != 64 && d != 128) || (chunk != 64 && chunk != 128) || L > kLongconvMaxL || short_width < 1 || short_width > 16)
        return CHELA_ERR_UNSUPPORTED;
    const MixerPlan p = mixer_plan(B, L, D, H, chunk, gated);
    if (!workspace || workspace_bytes < p.total) return CHELA_ERR_WORKSPACE;
    char *ws = (char *)workspace;
    float *z = (float *)(ws + p.off_z), *qq = (float *)(ws + p.off_q), *kk = (float *)(ws + p.off_k),
          *vv = (float *)(ws + p.off_v);
    const size_t M = (size_t)B * L;

    const size_t n = M * D;
    // gated form: the attention output goes to scratch, then u = o . G_a . G_o + x . (1 - G_o)  (Eqs. 8, 9, 13, 14)
    void *attn_out = gated ? (void *)(ws + p.off_o) : o;
    const chela_dtype_t attn_dtype = gated ? CHELA_F32 : out_dtype;
    // Tensor-core path: every intermediate (Z, Q, K, V) is a bf16 pair (hi + lo, about 16 mantissa bits) and
    // every product takes three tensor-core terms; single bf16 intermediates would cost the normalised
    // output its leading digits (cancellation in Q K^T on rows with a small pre-norm RMS).
    const bool tensor_path = in_dtype == CHELA_BF16 && (d == 64 || d == 128) &&
                             gemm_sm100_supported(M, D, D, CHELA_BF16_PAIR, CHELA_BF16, CHELA_BF16_PAIR);
    chela_status_t st;
    if (tensor_path) {
        __nv_bfloat16 *zp = (__nv_bfloat16 *)z, *qp = (__nv_bfloat16 *)qq, *kp = (__nv_bfloat16 *)kk, *vp = (__nv_bfloat16 *)vv;
        int *status = (int *)ws + 1;   // word 1 of the header: the GEMMs; word 0: the attention kernels
        // Z stays in the FFT kernel's row layout [B][D][L] when the projections can read it as a transposed operand:
        // saves the transpose back to token-major
        const int Ls = longconv_row_stride(L);
        const bool zt = !qk_diag && longconv_transposed_pair_supported(L) && gemm_sm100_at_supported(B, L, Ls, D, D);
        st = launch_longconv(x, k_long, w_short, short_width, zp, B, L, D, in_dtype, CHELA_BF16_PAIR, ws + p.off_conv, stream, zt, spectrum);
        if (st != CHELA_OK) return st;
        if (cudaMemsetAsync(status, 0, sizeof(int), stream) != cudaSuccess) return CHELA_ERR_CUDA;
        if (zt) {
            st = launch_gemm_sm100_at(zp, B, L, Ls, w_q, b_q, qp, D, D, 0, status, stream);
            if (st == CHELA_OK) st = launch_gemm_sm100_at(zp, B, L, Ls, w_k, b_k, kp, D, D, 0, status, stream);
        } else if (qk_diag) {
            st = launch_affine_pair(zp, w_q, b_q, qp, M, D, in_dtype, stream);
            if (st == CHELA_OK) st = launch_affine_pair(zp, w_k, b_k, kp, M, D, in_dtype, stream);
        } else {
            st = launch_gemm_sm100(zp, w_q, b_q, qp, M, D, D, 0, CHELA_BF16_PAIR, CHELA_BF16_PAIR, status, stream);
            if (st == CHELA_OK) st = launch_gemm_sm100(zp, w_k, b_k, kp, M, D, D, 0, CHELA_BF16_PAIR, CHELA_BF16_PAIR, status, stream);
        }
        if (st != CHELA_OK) return st;
        st = launch_gemm_sm100(x, w_v, b_v, vp, M, D, D, v_silu ? 1 : 0, CHELA_BF16, CHELA_BF16_PAIR, status, stream);
        if (st != CHELA_OK) return st;
        if (gated) {   // G_a = silu(Z W_a + b_a), G_o = sigmoid(Z W_o + b_o), as bf16 pairs
            if (zt) {
                st = launch_gemm_sm100_at(zp, B, L, Ls, w_a, b_a, ws + p.off_ga, D, D, 1, status, stream);
                if (st == CHELA_OK) st = launch_gemm_sm100_at(zp, B, L, Ls, w_o, b_o, ws + p.off_go, D, D, 2, status, stream);
            } else {
                st = launch_gemm_sm100(zp, w_a, b_a, ws + p.off_ga, M, D, D, 1, CHELA_BF16_PAIR, CHELA_BF16_PAIR, status, stream);
                if (st == CHELA_OK) st = launch_gemm_sm100(zp, w_o, b_o, ws + p.off_go, M, D, D, 2, CHELA_BF16_PAIR, CHELA_BF16_PAIR, status, stream);
            }
            if (st != CHELA_OK) return st;
        }
        st = launch_linattn_sm100(qp, kp, vp, attn_out, B, H, L, d, chunk, CHELA_BF16_PAIR, attn_dtype, (int)norm, norm_eps, 1.0f,
                                  ws + p.off_attn, stream);
        if (st != CHELA_OK || !gated) return st;
        return launch_gate_combine((const float *)attn_out, ws + p.off_ga, ws + p.off_go, CHELA_BF16_PAIR, x, in_dtype, o,
                                   out_dtype, n, stream);
    }
    // fp32 path.  Z = K_l(silu(K_s(X)))  (Eq. 7), kept in fp32
    st = launch_longconv(x, k_long, w_short, short_width, z, B, L, D, in_dtype, CHELA_F32,
                         ws + p.off_conv, stream, false, spectrum);
    if (st != CHELA_OK) return st;
    // Q, K from Z (Eqs. 10-11, or dense projections), V from X (Eq. 12)
    if (qk_diag) {
        st = launch_affine(z, w_q, b_q, qq, M, D, in_dtype, stream);
        if (st == CHELA_OK) st = launch_affine(z, w_k, b_k, kk, M, D, in_dtype, stream);
    } else {
        st = launch_gemm_simt(z, w_q, b_q, qq, M, D, D, 0, CHELA_F32, in_dtype, CHELA_F32, stream);
        if (st == CHELA_OK) st = launch_gemm_simt(z, w_k, b_k, kk, M, D, D, 0, CHELA_F32, in_dtype, CHELA_F32, stream);
    }
    if (st != CHELA_OK) return st;
    st = launch_gemm_simt(x, w_v, b_v, vv, M, D, D, v_silu ? 1 : 0, in_dtype, in_dtype, CHELA_F32, stream);
    if (st != CHELA_OK) return st;
    if (gated) {
        st = launch_gemm_simt(z, w_a, b_a, ws + p.off_ga, M, D, D, 1, CHELA_F32, in_dtype, CHELA_F32, stream);
        if (st == CHELA_OK) st = launch_gemm_simt(z, w_o, b_o, ws + p.off_go, M, D, D, 2, CHELA_F32, in_dtype, CHELA_F32, stream);
        if (st != CHELA_OK) return st;
    }
    // [B,L,D] with head h = columns [h*d,(h+1)*d) is [B,L,H,d]
    st = chela_linattn_fwd(qq, kk, vv, attn_out, B, H, L, d, d, chunk, CHELA_F32, attn_dtype, norm, norm_eps, 1.0f,
                           ws + p.off_attn, p.attn_bytes, stream);
    if (st != CHELA_OK || !gated) return st;
    return launch_gate_combine((const float *)attn_out, ws + p.off_ga, ws + p.off_go, CHELA_F32, x, in_dtype, o, out_dtype, n,
                               stream);
}
}  // namespace

extern "C" {

chela_status_t chela_mixer_fwd(const void *x, const float *w_short, int short_width, const float *k_long,
                               const void *w_q, const void *w_k, const void *w_v, const float *b_q,
                               const float *b_k, const float *b_v, int qk_diag, int v_silu, void *o, int B,
                               int L, int D, int H, int chunk, chela_dtype_t in_dtype,
                               chela_dtype_t out_dtype, chela_norm_t norm, float norm_eps, void *workspace,
                               size_t workspace_bytes, cudaStream_t stream)
{
    return mixer_impl(x, w_short, short_width, k_long, nullptr, w_q, w_k, w_v, b_q, b_k, b_v, nullptr, nullptr, nullptr, nullptr,
                      qk_diag, v_silu, o, B, L, D, H, chunk, in_dtype, out_dtype, norm, norm_eps, workspace, workspace_bytes,
                      stream);
}

chela_status_t chela_mixer_prepared_fwd(const void *x, const float *w_short, int short_width, const void *spectrum,
                                        const void *w_q, const void *w_k, const void *w_v, const float *b_q, const float *b_k,
                                        const float *b_v, const void *w_a, const float *b_a, const void *w_o, const float *b_o,
                                        int qk_diag, int v_silu, void *o, int B, int L, int D, int H, int chunk,
                                        chela_dtype_t in_dtype, chela_dtype_t out_dtype, chela_norm_t norm, float norm_eps,
                                        void *workspace, size_t workspace_bytes, cudaStream_t stream)
{
    if (!spectrum || (w_a != nullptr) != (w_o != nullptr)) return CHELA_ERR_INVALID_ARG;
    return mixer_impl(x, w_short, short_width, nullptr, spectrum, w_q, w_k, w_v, b_q, b_k, b_v, w_a, b_a, w_o, b_o, qk_diag, v_silu, o,
                      B, L, D, H, chunk, in_dtype, out_dtype, norm, norm_eps, workspace, workspace_bytes, stream);
}

chela_status_t chela_mixer_gated_fwd(const void *x, const float *w_short, int short_width, const float *k_long,
                                     const void *w_q, const void *w_k, const void *w_v, const float *b_q,
                                     const float *b_k, const float *b_v, const void *w_a, const float *b_a,
                                     const void *w_o, const float *b_o, int qk_diag, int v_silu, void *u, int B, int L,
                                     int D, int H, int chunk, chela_dtype_t in_dtype, chela_dtype_t out_dtype,
                                     chela_norm_t norm, float norm_eps, void *workspace, size_t workspace_bytes,
                                     cudaStream_t stream)
{
    if (!w_a || !w_o) return CHELA_ERR_INVALID_ARG;
    return mixer_impl(x, w_short, short_width, k_long, nullptr, w_q, w_k, w_v, b_q, b_k, b_v, w_a, b_a, w_o, b_o, qk_diag, v_silu, u,
                      B, L, D, H, chunk, in_dtype, out_dtype, norm, norm_eps, workspace, workspace_bytes, stream);
}

}  // extern "C"
