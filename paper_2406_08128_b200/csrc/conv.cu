// Short depthwise causal convolution + SiLU (Eq. 7, inner part) and the FFT long convolution
// (Eq. 6, Sec. 2.2).
//
// Long convolution pipeline (all fp32):
//   1. conv_transpose_kernel : x[B,L,D] -> a^T[B,D,Ls] fp32, applying the short convolution and
//      SiLU on the way when short taps are given (Eq. 7); rows become contiguous sequences.
//   2. twiddle_kernel        : w[j] = exp(-2 pi i j / N), j < M, N = 2M, M = nextpow2(L) (>= 16).
//   3. fft_conv_kernel (mode 0) : half spectrum K[c][0..M] of each zero-padded long kernel.
//   4. fft_conv_kernel (mode 1) : per (b,c) row, a real sequence of N = 2M samples (zero padded, so the
//      circular product is the causal linear convolution) is packed into M complex points,
//      transformed in shared memory (forward decimation-in-frequency, no reordering pass),
//      multiplied with the kernel spectrum, transformed back (decimation-in-time from
//      bit-reversed order) and written over its own row.
//   5. transpose_out_kernel  : z^T[B,D,Ls] -> z[B,L,D] in the output dtype.
#include "common.cuh"

namespace chela {
namespace {

// ------------------------------------------------------------------------------------ short conv

template <typename T>
__global__ void shortconv_kernel(const T *__restrict__ x, const float *__restrict__ w,
                                 const float *__restrict__ bias, T *__restrict__ y, int B, int L, int D,
                                 int width, int act)
{
    // one thread: 8 consecutive channels of one token; 128-bit accesses for bf16
    const size_t nvec = (size_t)B * L * (D / 8);
    for (size_t idx = blockIdx.x * (size_t)blockDim.x + threadIdx.x; idx < nvec;
         idx += (size_t)gridDim.x * blockDim.x) {
        const int cv = (int)(idx % (D / 8));
        const size_t bt = idx / (D / 8);
        const int t = (int)(bt % L);
        const int c0 = cv * 8;
        float acc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = bias ? bias[c0 + e] : 0.f;
        for (int j = 0; j < width && j <= t; ++j) {
            const T *px = x + (bt - j) * D + c0;
            const float4 lo = load4(px), hi = load4(px + 4);
            const float xv[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = fmaf(w[(c0 + e) * width + j], xv[e], acc[e]);
        }
        if (act) {
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = silu_f(acc[e]);
        }
        T *py = y + bt * D + c0;
        store4(py, make_float4(acc[0], acc[1], acc[2], acc[3]));
        store4(py + 4, make_float4(acc[4], acc[5], acc[6], acc[7]));
    }
}

// x[B,L,D] -> at[B,D,Ls] fp32; with taps: at = silu(shortconv(x)).  Tile: 32 channels x 64 tokens.
template <typename T>
__global__ void conv_transpose_kernel(const T *__restrict__ x, const float *__restrict__ w, int width,
                                      float *__restrict__ at, int L, int D, int Ls)
{
    __shared__ float tile[32][65];
    const int b = blockIdx.z, t0 = blockIdx.x * 64, c0 = blockIdx.y * 32;
    const int lane = threadIdx.x & 31, wrp = threadIdx.x >> 5;  // 256 threads = 8 warps
    const int c = c0 + lane;
    for (int tt = wrp; tt < 64; tt += 8) {
        const int t = t0 + tt;
        float acc = 0.f;
        if (t < L && c < D) {
            if (w) {
                for (int j = 0; j < width && j <= t; ++j)
                    acc = fmaf(w[c * width + j], load1(x + ((size_t)b * L + (t - j)) * D + c), acc);
                acc = silu_f(acc);
            } else {
                acc = load1(x + ((size_t)b * L + t) * D + c);
            }
        }
        tile[lane][tt] = acc;
    }
    __syncthreads();
    for (int cc = wrp; cc < 32; cc += 8) {
        if (c0 + cc >= D) continue;
        float *row = at + ((size_t)b * D + c0 + cc) * Ls;
        for (int tt = lane; tt < 64; tt += 32)
            if (t0 + tt < Ls) row[t0 + tt] = (t0 + tt < L) ? tile[cc][tt] : 0.f;
    }
}

// zt[B,D,Ls] fp32 -> z[B,L,D].  Tile: 64 channels x 32 tokens.
// lo_offset != 0: z is a bf16 pair; the low plane (z + lo_offset) receives round(value - high part).
template <typename T>
__global__ void transpose_out_kernel(const float *__restrict__ zt, T *__restrict__ z, int L, int D, int Ls, size_t lo_offset)
{
    __shared__ float tile[64][33];
    const int b = blockIdx.z, t0 = blockIdx.x * 32, c0 = blockIdx.y * 64;
    const int lane = threadIdx.x & 31, wrp = threadIdx.x >> 5;
    for (int cc = wrp; cc < 64; cc += 8) {
        const int c = c0 + cc, t = t0 + lane;
        tile[cc][lane] = (c < D && t < L) ? zt[((size_t)b * D + c) * Ls + t] : 0.f;
    }
    __syncthreads();
    for (int tt = wrp; tt < 32; tt += 8) {
        const int t = t0 + tt;
        if (t >= L) continue;
        for (int cc = lane; cc < 64; cc += 32)
            if (c0 + cc < D) {
                const size_t idx = ((size_t)b * L + t) * D + c0 + cc;
                const float val = tile[cc][tt];
                store1(z + idx, val);
                if (lo_offset) store1(z + lo_offset + idx, val - load1(z + idx));
            }
    }
}

// ------------------------------------------------------------------------------------ FFT pieces

__global__ void twiddle_kernel(float2 *__restrict__ tw, int M)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j < M) {
        double s, c;
        sincospi(-(double)j / (double)M, &s, &c);  // exp(-2 pi i j / (2M))
        tw[j] = make_float2((float)c, (float)s);
    }
}

__device__ __forceinline__ float2 cmul(float2 a, float2 b) { return make_float2(a.x * b.x - a.y * b.y, a.x * b.y + a.y * b.x); }
__device__ __forceinline__ float2 cmulc(float2 a, float2 b) { return make_float2(a.x * b.x + a.y * b.y, a.y * b.x - a.x * b.y); }  // a * conj(b)
__device__ __forceinline__ float2 cadd(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ float2 csub(float2 a, float2 b) { return make_float2(a.x - b.x, a.y - b.y); }
__device__ __forceinline__ float2 cconj(float2 a) { return make_float2(a.x, -a.y); }

// Forward M-point FFT in shared memory, decimation in frequency: natural order in, bit-reversed
// order out.  tw[j] = exp(-2 pi i j / (2M)), so exp(-2 pi i k / len) = tw[k * (2M / len)].
__device__ void fft_forward_dif(float2 *s, const float2 *__restrict__ tw, int M, int logM)
{
    int len = M, st = 2;  // st = 2M / len
    int stages = logM;
    for (; stages >= 2; stages -= 2, len >>= 2, st <<= 2) {
        const int quarter = len >> 2;
        for (int g = threadIdx.x; g < (M >> 2); g += blockDim.x) {
            const int k = g & (quarter - 1);
            const int i0 = ((g - k) << 2) + k;
            float2 a = s[i0], b = s[i0 + quarter], c = s[i0 + 2 * quarter], d = s[i0 + 3 * quarter];
            // stage "len": pairs (a,c) twiddle k, (b,d) twiddle k + quarter
            float2 a1 = cadd(a, c), c1 = cmul(csub(a, c), tw[k * st]);
            float2 b1 = cadd(b, d), d1 = cmul(csub(b, d), tw[(k + quarter) * st]);
            // stage "len/2": pairs (a1,b1) and (c1,d1), both twiddle k (at stride 2*st)
            const float2 w2 = tw[k * 2 * st];
            s[i0] = cadd(a1, b1);
            s[i0 + quarter] = cmul(csub(a1, b1), w2);
            s[i0 + 2 * quarter] = cadd(c1, d1);
            s[i0 + 3 * quarter] = cmul(csub(c1, d1), w2);
        }
        __syncthreads();
    }
    if (stages == 1) {  // len == 2
        for (int g = threadIdx.x; g < (M >> 1); g += blockDim.x) {
            float2 a = s[2 * g], b = s[2 * g + 1];
            s[2 * g] = cadd(a, b);
            s[2 * g + 1] = csub(a, b);
        }
        __syncthreads();
    }
}

// Inverse (unscaled) M-point FFT, decimation in time: bit-reversed order in, natural order out.
__device__ void fft_inverse_dit(float2 *s, const float2 *__restrict__ tw, int M, int logM)
{
    int len = 2;
    int stages = logM;
    if (stages & 1) {
        for (int g = threadIdx.x; g < (M >> 1); g += blockDim.x) {
            float2 a = s[2 * g], b = s[2 * g + 1];
            s[2 * g] = cadd(a, b);
            s[2 * g + 1] = csub(a, b);
        }
        __syncthreads();
        len = 4;
        --stages;
    }
    // fused pairs of stages: first "len", then "2*len"
    for (; stages >= 2; stages -= 2, len <<= 2) {
        const int half = len >> 1;          // butterfly span of the first stage
        const int st1 = (2 * M) / len;      // twiddle stride of the first stage
        const int st2 = st1 >> 1;           // of the second stage (length 2*len)
        for (int g = threadIdx.x; g < (M >> 2); g += blockDim.x) {
            const int k = g & (half - 1);
            const int i0 = ((g - k) << 2) + k;
            float2 a = s[i0], b = s[i0 + half], c = s[i0 + 2 * half], d = s[i0 + 3 * half];
            // first stage (length len): pairs (a,b) and (c,d), twiddle conj(w_len^k)
            const float2 w1 = tw[k * st1];
            const float2 bt = cmulc(b, w1), dt = cmulc(d, w1);
            const float2 a1 = cadd(a, bt), b1 = csub(a, bt), c1 = cadd(c, dt), d1 = csub(c, dt);
            // second stage (length 2*len): pairs (a1,c1) twiddle k, (b1,d1) twiddle k + half
            const float2 ct = cmulc(c1, tw[k * st2]), dtt = cmulc(d1, tw[(k + half) * st2]);
            s[i0] = cadd(a1, ct);
            s[i0 + 2 * half] = csub(a1, ct);
            s[i0 + half] = cadd(b1, dtt);
            s[i0 + 3 * half] = csub(b1, dtt);
        }
        __syncthreads();
    }
}

__device__ __forceinline__ int bitrev(int f, int logM) { return (int)(__brev((unsigned)f) >> (32 - logM)); }

// mode 0: rows = long kernels k[D][L] (row stride L), writes the half spectrum spec[row][0..M].
// mode 1: rows = sequences at[B*D][Ls]; multiplies with spec[row % D] and writes the causal
//         convolution back over the row.
template <int MODE>
__global__ void fft_conv_kernel(float *__restrict__ rows, int row_stride, int L, int D, int M, int logM,
                                const float2 *__restrict__ tw, float2 *__restrict__ spec)
{
    extern __shared__ __align__(16) float2 s[];
    const int row = blockIdx.x;
    float *x = rows + (size_t)row * row_stride;
    // pack: s[n] = x[2n] + i x[2n+1], zero beyond L
    for (int n = threadIdx.x; n < M; n += blockDim.x) {
        const int t = 2 * n;
        float re = 0.f, im = 0.f;
        if (MODE == 1) {  // padded, 8-byte aligned rows
            if (t + 1 < L) {
                const float2 p = *reinterpret_cast<const float2 *>(x + t);
                re = p.x; im = p.y;
            } else if (t < L) re = x[t];
        } else {
            if (t < L) re = x[t];
            if (t + 1 < L) im = x[t + 1];
        }
        s[n] = make_float2(re, im);
    }
    __syncthreads();
    fft_forward_dif(s, tw, M, logM);
    // C[f] sits at s[bitrev(f)].  Spectrum of the real length-2M sequence:
    //   E = (C[f] + conj C[M-f]) / 2, O = -i (C[f] - conj C[M-f]) / 2,
    //   X[f] = E + w^f O,  X[M-f] = conj(E - w^f O),  w = exp(-2 pi i / 2M); X[M] = E[0] - O[0].
    float2 *kspec = spec + (size_t)(MODE == 1 ? row % D : row) * (M + 1);
    for (int f = threadIdx.x; f <= (M >> 1); f += blockDim.x) {
        const int pf = bitrev(f, logM), pm = bitrev((M - f) & (M - 1), logM);
        const float2 Cf = s[pf], Cm = s[pm];
        const float2 E = make_float2(0.5f * (Cf.x + Cm.x), 0.5f * (Cf.y - Cm.y));
        const float2 O = make_float2(0.5f * (Cf.y + Cm.y), -0.5f * (Cf.x - Cm.x));
        const float2 wO = cmul(tw[f], O);
        float2 Xf = cadd(E, wO), Xm = cconj(csub(E, wO));
        if (MODE == 0) {
            if (f == 0) {
                kspec[0] = make_float2(E.x + O.x, 0.f);
                kspec[M] = make_float2(E.x - O.x, 0.f);
            } else {
                kspec[f] = Xf;
                kspec[M - f] = Xm;
            }
        } else {
            // Y = X K, then the packed spectrum of y: C'[f] = E' + i O',
            //   E' = (Y[f] + conj Y[M-f]) / 2,  O' = (Y[f] - conj Y[M-f]) / 2 * conj(w^f),
            //   C'[M-f] = conj(E') + i conj(O').
            float2 Yf, Ym;
            if (f == 0) {
                Yf = make_float2((E.x + O.x) * kspec[0].x, 0.f);
                Ym = make_float2((E.x - O.x) * kspec[M].x, 0.f);
            } else {
                Yf = cmul(Xf, kspec[f]);
                Ym = cmul(Xm, kspec[M - f]);
            }
            const float2 Ep = make_float2(0.5f * (Yf.x + Ym.x), 0.5f * (Yf.y - Ym.y));
            const float2 Dp = make_float2(0.5f * (Yf.x - Ym.x), 0.5f * (Yf.y + Ym.y));
            const float2 Op = cmulc(Dp, tw[f]);
            s[pf] = make_float2(Ep.x - Op.y, Ep.y + Op.x);          // E' + i O'
            if (pm != pf) s[pm] = make_float2(Ep.x + Op.y, -Ep.y + Op.x);  // conj(E') + i conj(O')
        }
    }
    if (MODE == 0) return;
    __syncthreads();
    fft_inverse_dit(s, tw, M, logM);
    const float inv = 1.0f / (float)M;
    for (int n = threadIdx.x; 2 * n < row_stride; n += blockDim.x) {
        const int t = 2 * n;
        float2 p = (n < M) ? s[n] : make_float2(0.f, 0.f);
        p.x = (t < L) ? p.x * inv : 0.f;
        p.y = (t + 1 < L) ? p.y * inv : 0.f;
        *reinterpret_cast<float2 *>(x + t) = p;
    }
}

}  // namespace

chela_status_t launch_shortconv(const void *x, const float *w, const float *bias, void *y, int B, int L,
                                int D, int width, int act, chela_dtype_t io_dtype, cudaStream_t stream)
{
    const size_t nvec = (size_t)B * L * (D / 8);
    const int threads = 256;
    const int blocks = (int)((nvec + threads - 1) / threads < (size_t)148 * 32 ? (nvec + threads - 1) / threads
                                                                                : (size_t)148 * 32);
    if (io_dtype == CHELA_BF16)
        shortconv_kernel<__nv_bfloat16><<<blocks, threads, 0, stream>>>((const __nv_bfloat16 *)x, w, bias,
                                                                        (__nv_bfloat16 *)y, B, L, D, width, act);
    else
        shortconv_kernel<float><<<blocks, threads, 0, stream>>>((const float *)x, w, bias, (float *)y, B, L, D,
                                                                width, act);
    return last_launch_status();
}

namespace {
struct LongconvPlan {
    int M, logM, Ls;
    size_t off_at, off_tw, off_spec, total;
};
LongconvPlan longconv_plan(int B, int L, int D)
{
    LongconvPlan p;
    p.M = next_pow2(L) < 16 ? 16 : next_pow2(L);
    p.logM = 0;
    while ((1 << p.logM) < p.M) ++p.logM;
    p.Ls = (int)align_up((size_t)L, 8);
    p.off_at = 0;
    p.off_tw = align_up(p.off_at + (size_t)B * D * p.Ls * sizeof(float), 256);
    p.off_spec = align_up(p.off_tw + (size_t)p.M * sizeof(float2), 256);
    p.total = align_up(p.off_spec + (size_t)D * (p.M + 1) * sizeof(float2), 256);
    return p;
}
}  // namespace

size_t longconv_workspace_bytes(int B, int L, int D) { return longconv_plan(B, L, D).total; }

chela_status_t launch_longconv(const void *x, const float *k_long, const float *w_short, int short_width,
                               void *z, int B, int L, int D, chela_dtype_t in_dtype,
                               chela_dtype_t out_dtype, void *workspace, cudaStream_t stream)
{
    const LongconvPlan p = longconv_plan(B, L, D);
    char *ws = (char *)workspace;
    float *at = (float *)(ws + p.off_at);
    float2 *tw = (float2 *)(ws + p.off_tw);
    float2 *spec = (float2 *)(ws + p.off_spec);

    dim3 g1((L + 63) / 64, (D + 31) / 32, B);
    if (in_dtype == CHELA_BF16)
        conv_transpose_kernel<__nv_bfloat16><<<g1, 256, 0, stream>>>((const __nv_bfloat16 *)x, w_short, short_width,
                                                                     at, L, D, p.Ls);
    else
        conv_transpose_kernel<float><<<g1, 256, 0, stream>>>((const float *)x, w_short, short_width, at, L, D, p.Ls);
    twiddle_kernel<<<(p.M + 255) / 256, 256, 0, stream>>>(tw, p.M);

    const size_t smem = (size_t)p.M * sizeof(float2);
    int threads = p.M / 4;
    threads = threads < 32 ? 32 : (threads > 1024 ? 1024 : threads);
    cudaError_t e = cudaFuncSetAttribute(fft_conv_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(fft_conv_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return CHELA_ERR_CUDA;
    fft_conv_kernel<0><<<D, threads, smem, stream>>>(const_cast<float *>(k_long), L, L, D, p.M, p.logM, tw, spec);
    fft_conv_kernel<1><<<B * D, threads, smem, stream>>>(at, p.Ls, L, D, p.M, p.logM, tw, spec);

    dim3 g2((L + 31) / 32, (D + 63) / 64, B);
    if (out_dtype == CHELA_BF16 || out_dtype == CHELA_BF16_PAIR)
        transpose_out_kernel<__nv_bfloat16><<<g2, 256, 0, stream>>>(at, (__nv_bfloat16 *)z, L, D, p.Ls,
                                                                    out_dtype == CHELA_BF16_PAIR ? (size_t)B * L * D : 0);
    else
        transpose_out_kernel<float><<<g2, 256, 0, stream>>>(at, (float *)z, L, D, p.Ls, 0);
    return last_launch_status();
}

}  // namespace chela
