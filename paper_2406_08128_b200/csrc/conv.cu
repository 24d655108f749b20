// Short depthwise causal convolution + SiLU (Eq. 7, inner part) and the FFT long convolution
// (Eq. 6, Sec. 2.2).
//
// Long convolution pipeline (all fp32):
//   1. conv_transpose_kernel : x[B,L,D] -> a^T[B,D,Ls] fp32, applying the short convolution and
//      SiLU on the way when short taps are given (Eq. 7); rows become contiguous sequences.
//   2. twiddle_kernel        : w[j] = exp(-2 pi i j / N), j < M, N = 2M, M = nextpow2(L) (>= 16).
//   3. FFT kernel, mode 0   : half spectrum K[c][0..M] of each zero-padded long kernel.
//   4. FFT kernel, mode 1   : per (b,c) row, a real sequence of N = 2M samples (zero padded, so the
//      circular product is the causal linear convolution) is packed into M complex points,
//      transformed in shared memory (forward decimation-in-frequency, no reordering pass),
//      multiplied with the kernel spectrum, transformed back (decimation-in-time from
//      bit-reversed order) and written over its own row.
//   5. transpose_out_kernel  : z^T[B,D,Ls] -> z[B,L,D] in the output dtype.
// Steps 3 and 4 run fft_conv_fast_kernel (longconv_fft.cu: compile-time strides) for M = 2^10 .. 2^14 and the
// generic fft_conv_kernel of this file for every other size.
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

// Fast form for W <= 4 taps: one thread owns CH consecutive channels (CH = 4: one 8-byte access for bf16) and
// kTok consecutive tokens, kSub at a time (kSub loads in flight), with the taps and the previous W-1 inputs in
// registers: every input is loaded once plus a W-1 token halo per thread.  CH = 4 keeps the thread at about 64
// registers (four CTAs per SM); with 8 channels it needed 121 and the kernel ran at a third of the HBM rate.
template <typename T, int W, int CH>
__global__ void __launch_bounds__(256, 4)
shortconv_fast_kernel(const T *__restrict__ x, const float *__restrict__ w, const float *__restrict__ bias,
                      T *__restrict__ y, int B, int L, int D, int act)
{
    constexpr int kTok = 32, kSub = 4;
    const int nvec = D / CH, nblk = (L + kTok - 1) / kTok;
    const size_t total = (size_t)B * nblk * nvec;
    for (size_t idx = blockIdx.x * (size_t)blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
        const int cv = (int)(idx % nvec);
        const size_t r = idx / nvec;
        const int tb = (int)(r % nblk), b = (int)(r / nblk);
        const int c0 = cv * CH, t0 = tb * kTok;
        float wt[CH][W], bs[CH];
#pragma unroll
        for (int e = 0; e < CH; ++e) {
            bs[e] = bias ? bias[c0 + e] : 0.f;
#pragma unroll
            for (int j = 0; j < W; ++j) wt[e][j] = w[(c0 + e) * W + j];
        }
        // xin[i] = x[ts - (W-1) + i] for the current sub-block of kSub tokens starting at ts
        float xin[kSub + W - 1][CH];
        auto load = [&](int t, float (&dst)[CH]) {
            if (t < 0 || t >= L) {
#pragma unroll
                for (int e = 0; e < CH; ++e) dst[e] = 0.f;
                return;
            }
            const T *px = x + ((size_t)b * L + t) * D + c0;
#pragma unroll
            for (int v4 = 0; v4 < CH / 4; ++v4) {
                const float4 f = load4(px + 4 * v4);
                dst[4 * v4] = f.x; dst[4 * v4 + 1] = f.y; dst[4 * v4 + 2] = f.z; dst[4 * v4 + 3] = f.w;
            }
        };
#pragma unroll
        for (int i = 0; i < W - 1; ++i) load(t0 - (W - 1) + i, xin[i]);
#pragma unroll 1
        for (int sb = 0; sb < kTok / kSub; ++sb) {
            const int ts = t0 + sb * kSub;
            if (ts >= L) break;
#pragma unroll
            for (int i = 0; i < kSub; ++i) load(ts + i, xin[W - 1 + i]);   // kSub loads in flight
#pragma unroll
            for (int i = 0; i < kSub; ++i) {
                if (ts + i >= L) break;
                float acc[CH];
#pragma unroll
                for (int e = 0; e < CH; ++e) {
                    acc[e] = bs[e];
#pragma unroll
                    for (int j = 0; j < W; ++j) acc[e] = fmaf(wt[e][j], xin[i + W - 1 - j][e], acc[e]);
                    if (act) acc[e] = silu_f(acc[e]);
                }
                T *py = y + ((size_t)b * L + ts + i) * D + c0;
#pragma unroll
                for (int v4 = 0; v4 < CH / 4; ++v4)
                    store4(py + 4 * v4, make_float4(acc[4 * v4], acc[4 * v4 + 1], acc[4 * v4 + 2], acc[4 * v4 + 3]));
            }
#pragma unroll
            for (int i = 0; i < W - 1; ++i)
#pragma unroll
                for (int e = 0; e < CH; ++e) xin[i][e] = xin[kSub + i][e];
        }
    }
}

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

// Fast form of conv_transpose_kernel for bf16 input and W <= 4 taps (W = 0: plain transpose): a
// 64-channel x 64-token tile; each lane owns two adjacent channels (4-byte loads, 128 B per warp row) and
// walks 8 consecutive tokens with the previous W-1 inputs in registers.
template <int W>
__global__ void __launch_bounds__(256)
conv_transpose_bf16_kernel(const __nv_bfloat16 *__restrict__ x, const float *__restrict__ w, float *__restrict__ at, int L,
                           int D, int Ls)
{
    __shared__ float tile[64][65];
    const int b = blockIdx.z, t0 = blockIdx.x * 64, c0 = blockIdx.y * 64;
    const int lane = threadIdx.x & 31, wrp = threadIdx.x >> 5;
    const int c = c0 + 2 * lane;
    constexpr int WW = W > 0 ? W : 1;
    float w0[WW], w1[WW];
#pragma unroll
    for (int j = 0; j < WW; ++j) {
        w0[j] = (W > 0 && c < D) ? w[c * W + j] : 0.f;
        w1[j] = (W > 0 && c + 1 < D) ? w[(c + 1) * W + j] : 0.f;
    }
    float2 hist[WW];   // hist[j] = x[t - j]
#pragma unroll
    for (int j = 0; j < WW; ++j) hist[j] = make_float2(0.f, 0.f);
    const int ts = t0 + wrp * 8;
    auto load = [&](int t) -> float2 {
        if (t < 0 || t >= L || c >= D) return make_float2(0.f, 0.f);   // D is even: c + 1 < D whenever c < D
        return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(x + ((size_t)b * L + t) * D + c));
    };
#pragma unroll
    for (int j = 1; j < WW; ++j) hist[j] = load(ts - j);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        hist[0] = load(ts + i);
        float2 y;
        if (W > 0) {
            y = make_float2(0.f, 0.f);
#pragma unroll
            for (int j = 0; j < WW; ++j) {
                y.x = fmaf(w0[j], hist[j].x, y.x);
                y.y = fmaf(w1[j], hist[j].y, y.y);
            }
            y.x = silu_f(y.x);
            y.y = silu_f(y.y);
        } else {
            y = hist[0];
        }
        tile[2 * lane][wrp * 8 + i] = y.x;
        tile[2 * lane + 1][wrp * 8 + i] = y.y;
#pragma unroll
        for (int j = WW - 1; j > 0; --j) hist[j] = hist[j - 1];
    }
    __syncthreads();
    // rows of at: 64 tokens = 256 B per channel; a half-warp writes one row with float4 stores
    const int half = lane >> 4, l16 = lane & 15;
    for (int cc = wrp * 2 + half; cc < 64; cc += 16) {
        if (c0 + cc >= D) continue;
        const int t = t0 + 4 * l16;
        if (t >= Ls) continue;   // Ls is a multiple of 8: a float4 is either inside or outside
        float4 v = make_float4(tile[cc][4 * l16], tile[cc][4 * l16 + 1], tile[cc][4 * l16 + 2], tile[cc][4 * l16 + 3]);
        if (t + 0 >= L) v.x = 0.f;
        if (t + 1 >= L) v.y = 0.f;
        if (t + 2 >= L) v.z = 0.f;
        if (t + 3 >= L) v.w = 0.f;
        *reinterpret_cast<float4 *>(at + ((size_t)b * D + c0 + cc) * Ls + t) = v;
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

// Fast form for bf16 (pair) output: 64 channels x 64 tokens; float4 loads along tokens, 4-byte stores of
// two adjacent channels (128 B per warp row).
__global__ void __launch_bounds__(256)
transpose_out_bf16_kernel(const float *__restrict__ zt, __nv_bfloat16 *__restrict__ z, int L, int D, int Ls, size_t lo_offset)
{
    __shared__ float tile[64][65];
    const int b = blockIdx.z, t0 = blockIdx.x * 64, c0 = blockIdx.y * 64;
    const int lane = threadIdx.x & 31, wrp = threadIdx.x >> 5;
    const int half = lane >> 4, l16 = lane & 15;
    for (int cc = wrp * 2 + half; cc < 64; cc += 16) {
        const int t = t0 + 4 * l16;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c0 + cc < D && t < Ls) v = *reinterpret_cast<const float4 *>(zt + ((size_t)b * D + c0 + cc) * Ls + t);
        tile[cc][4 * l16] = v.x;
        tile[cc][4 * l16 + 1] = v.y;
        tile[cc][4 * l16 + 2] = v.z;
        tile[cc][4 * l16 + 3] = v.w;
    }
    __syncthreads();
    const int c = c0 + 2 * lane;
    if (c >= D) return;
    for (int tt = wrp; tt < 64; tt += 8) {
        const int t = t0 + tt;
        if (t >= L) break;
        const float v0 = tile[2 * lane][tt], v1 = tile[2 * lane + 1][tt];
        const __nv_bfloat162 hi = __floats2bfloat162_rn(v0, v1);
        const size_t idx = ((size_t)b * L + t) * D + c;
        *reinterpret_cast<__nv_bfloat162 *>(z + idx) = hi;
        if (lo_offset) {
            const float2 hf = __bfloat1622float2(hi);
            *reinterpret_cast<__nv_bfloat162 *>(z + lo_offset + idx) = __floats2bfloat162_rn(v0 - hf.x, v1 - hf.y);
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

// ---- in-shared-memory FFT: up to four radix-2 stages fused per pass in registers ---------------------
//
// Element e of the M-point array lives at phys(e): 16-byte chunks (two complex values) are XOR-swizzled
// inside groups of eight, so both access patterns of the passes are free of bank conflicts: lanes
// reading consecutive elements, and lanes reading 16 consecutive elements each (the contiguous pass).
__device__ __forceinline__ int phys(int e)
{
    const int c = e >> 1;
    return ((c ^ ((c >> 3) & 7)) << 1) | (e & 1);
}

// exp(-2 pi i m / 16), m = 0..7
__device__ __forceinline__ float2 root16(int m)
{
    switch (m) {
        case 0: return make_float2(1.f, 0.f);
        case 1: return make_float2(0.92387953251128674f, -0.38268343236508977f);
        case 2: return make_float2(0.70710678118654752f, -0.70710678118654752f);
        case 3: return make_float2(0.38268343236508977f, -0.92387953251128674f);
        case 4: return make_float2(0.f, -1.f);
        case 5: return make_float2(-0.38268343236508977f, -0.92387953251128674f);
        case 6: return make_float2(-0.70710678118654752f, -0.70710678118654752f);
        default: return make_float2(-0.92387953251128674f, -0.38268343236508977f);
    }
}

// Two-level twiddle table in shared memory: exp(-2 pi i j / 2M) = T1[j & 127] * T2[j >> 7], j < M.
struct Twiddles {
    const float2 *t1, *t2;
    __device__ __forceinline__ float2 operator()(int j) const { return cmul(t1[j & 127], t2[j >> 7]); }
};

// One decimation-in-frequency pass: R radix-2 stages of sub-lengths len, len/2, ..., fused on the 2^R
// elements i0 + j * (len >> R) that they keep among themselves.  In place; after all passes element
// of frequency f sits at the bit-reversed position.
template <int R, bool kContiguous>
__device__ __forceinline__ void dif_pass(float2 *s, const Twiddles &tw, int M, int len)
{
    constexpr int G = 1 << R;
    const int q = len >> R, tws = (2 * M) / len;
    // a stride of whole 128-element blocks leaves the swizzle pattern of the group's elements unchanged
    const bool aligned = (q & 127) == 0;
    for (int g = threadIdx.x; g < (M >> R); g += blockDim.x) {
        const int k = g & (q - 1);
        const int i0 = ((g - k) << R) + k;
        const int p0 = phys(i0);
        float2 v[G];
        if (kContiguous) {   // q == 1, G == 16: eight 16-byte chunks per thread
#pragma unroll
            for (int c = 0; c < G / 2; ++c) {
                const float4 t = *reinterpret_cast<const float4 *>(s + phys(i0 + 2 * c));
                v[2 * c] = make_float2(t.x, t.y);
                v[2 * c + 1] = make_float2(t.z, t.w);
            }
        } else if (aligned) {
#pragma unroll
            for (int j = 0; j < G; ++j) v[j] = s[p0 + j * q];
        } else {
#pragma unroll
            for (int j = 0; j < G; ++j) v[j] = s[phys(i0 + j * q)];
        }
#pragma unroll
        for (int st = 0; st < R; ++st) {
            const int h = G >> (st + 1);
            // W_len^(k 2^st): base twiddle of this stage; the rest of the exponent is a 16th root of unity
            const float2 wb = kContiguous ? make_float2(1.f, 0.f) : tw((k << st) * tws);
#pragma unroll
            for (int blk = 0; blk < (1 << st); ++blk)
#pragma unroll
                for (int jj = 0; jj < h; ++jj) {
                    const int ia = blk * 2 * h + jj, ib = ia + h;
                    const float2 a = v[ia], b = v[ib];
                    v[ia] = cadd(a, b);
                    const float2 w = (jj == 0) ? wb : (kContiguous ? root16((jj << st) * (16 / G)) : cmul(wb, root16((jj << st) * (16 / G))));
                    v[ib] = (kContiguous && jj == 0) ? csub(a, b) : cmul(csub(a, b), w);
                }
        }
        if (kContiguous) {
#pragma unroll
            for (int c = 0; c < G / 2; ++c)
                *reinterpret_cast<float4 *>(s + phys(i0 + 2 * c)) = make_float4(v[2 * c].x, v[2 * c].y, v[2 * c + 1].x, v[2 * c + 1].y);
        } else if (aligned) {
#pragma unroll
            for (int j = 0; j < G; ++j) s[p0 + j * q] = v[j];
        } else {
#pragma unroll
            for (int j = 0; j < G; ++j) s[phys(i0 + j * q)] = v[j];
        }
    }
    __syncthreads();
}

// One decimation-in-time pass of the inverse transform: R stages of sub-lengths len0, 2 len0, ..., on the
// 2^R elements i0 + j * (len0 / 2).  Consumes the bit-reversed order the forward passes leave.
template <int R, bool kContiguous>
__device__ __forceinline__ void dit_pass(float2 *s, const Twiddles &tw, int M, int len0)
{
    constexpr int G = 1 << R;
    const int h0 = len0 >> 1;
    const bool aligned = (h0 & 127) == 0;
    for (int g = threadIdx.x; g < (M >> R); g += blockDim.x) {
        const int k = g & (h0 - 1);
        const int i0 = ((g - k) << R) + k;
        const int p0 = phys(i0);
        float2 v[G];
        if (kContiguous) {   // len0 == 2, G == 16
#pragma unroll
            for (int c = 0; c < G / 2; ++c) {
                const float4 t = *reinterpret_cast<const float4 *>(s + phys(i0 + 2 * c));
                v[2 * c] = make_float2(t.x, t.y);
                v[2 * c + 1] = make_float2(t.z, t.w);
            }
        } else if (aligned) {
#pragma unroll
            for (int j = 0; j < G; ++j) v[j] = s[p0 + j * h0];
        } else {
#pragma unroll
            for (int j = 0; j < G; ++j) v[j] = s[phys(i0 + j * h0)];
        }
#pragma unroll
        for (int st = 0; st < R; ++st) {
            const int d = 1 << st;
            const float2 wb = kContiguous ? make_float2(1.f, 0.f) : tw(k * ((2 * M) / (len0 << st)));
#pragma unroll
            for (int j = 0; j < G; ++j) {
                if (j & d) continue;
                const int jj = j & (d - 1);
                const float2 a = v[j];
                float2 bt;
                if (kContiguous && jj == 0) bt = v[j + d];
                else {
                    const float2 w = (jj == 0) ? wb : (kContiguous ? root16(jj * (16 >> (st + 1))) : cmul(wb, root16(jj * (16 >> (st + 1)))));
                    bt = cmulc(v[j + d], w);
                }
                v[j] = cadd(a, bt);
                v[j + d] = csub(a, bt);
            }
        }
        if (kContiguous) {
#pragma unroll
            for (int c = 0; c < G / 2; ++c)
                *reinterpret_cast<float4 *>(s + phys(i0 + 2 * c)) = make_float4(v[2 * c].x, v[2 * c].y, v[2 * c + 1].x, v[2 * c + 1].y);
        } else if (aligned) {
#pragma unroll
            for (int j = 0; j < G; ++j) s[p0 + j * h0] = v[j];
        } else {
#pragma unroll
            for (int j = 0; j < G; ++j) s[phys(i0 + j * h0)] = v[j];
        }
    }
    __syncthreads();
}

template <bool kForward>
__device__ __forceinline__ void pass_r(int R, float2 *s, const Twiddles &tw, int M, int len)
{
    if (kForward) {
        if (R == 1) dif_pass<1, false>(s, tw, M, len);
        else if (R == 2) dif_pass<2, false>(s, tw, M, len);
        else if (R == 3) dif_pass<3, false>(s, tw, M, len);
        else dif_pass<4, false>(s, tw, M, len);
    } else {
        if (R == 1) dit_pass<1, false>(s, tw, M, len);
        else if (R == 2) dit_pass<2, false>(s, tw, M, len);
        else if (R == 3) dit_pass<3, false>(s, tw, M, len);
        else dit_pass<4, false>(s, tw, M, len);
    }
}

// Forward M-point FFT (M >= 16): natural order in, bit-reversed order out.  Stages are grouped
// r0, 4, 4, ..., 4 with r0 = logM mod 4 (4 if that is 0); the last pass works on 16 contiguous elements.
__device__ void fft_forward_dif(float2 *s, const Twiddles &tw, int M, int logM)
{
    const int r0 = ((logM - 1) & 3) + 1;
    int len = M;
    if (logM > 4) {
        pass_r<true>(r0, s, tw, M, len);
        len >>= r0;
        for (; len > 16; len >>= 4) dif_pass<4, false>(s, tw, M, len);
    }
    dif_pass<4, true>(s, tw, M, 16);
}

// Inverse (unscaled) M-point FFT: bit-reversed order in, natural order out (mirror of the forward passes).
__device__ void fft_inverse_dit(float2 *s, const Twiddles &tw, int M, int logM)
{
    const int r0 = ((logM - 1) & 3) + 1;
    dit_pass<4, true>(s, tw, M, 2);
    if (logM > 4) {
        int len0 = 32;
        for (; (len0 << 3) <= (M >> r0); len0 <<= 4) dit_pass<4, false>(s, tw, M, len0);
        pass_r<false>(r0, s, tw, M, len0);
    }
}

__device__ __forceinline__ int bitrev(int f, int logM) { return (int)(__brev((unsigned)f) >> (32 - logM)); }

// mode 0: rows = long kernels k[D][L] (row stride L), writes the half spectrum spec[row][0..M].
// mode 1: rows = sequences at[B*D][Ls]; multiplies with spec[row % D] and writes the causal
//         convolution back over the row.
template <int MODE>
__global__ void __launch_bounds__(1024) fft_conv_kernel(float *__restrict__ rows, int row_stride, int L, int D, int M, int logM,
                                const float2 *__restrict__ tw_global, float2 *__restrict__ spec, int spec_stride)
{
    extern __shared__ __align__(16) float2 s[];   // M data points (swizzled), then the two twiddle tables
    float2 *t1 = s + M, *t2 = t1 + 128;
    for (int j = threadIdx.x; j < 128; j += blockDim.x) {
        t1[j] = (j < M) ? tw_global[j] : make_float2(1.f, 0.f);
        t2[j] = (128 * j < M) ? tw_global[128 * j] : make_float2(1.f, 0.f);
    }
    const Twiddles tw = {t1, t2};
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
        s[phys(n)] = make_float2(re, im);
    }
    __syncthreads();
    fft_forward_dif(s, tw, M, logM);
    // C[f] sits at s[bitrev(f)].  Spectrum of the real length-2M sequence:
    //   E = (C[f] + conj C[M-f]) / 2, O = -i (C[f] - conj C[M-f]) / 2,
    //   X[f] = E + w^f O,  X[M-f] = conj(E - w^f O),  w = exp(-2 pi i / 2M); X[M] = E[0] - O[0].
    // The kernel spectrum is kept in the same bit-reversed order as the data (entry p holds K[bitrev(p)];
    // entry M holds the Nyquist term), and the loop runs over positions p rather than frequencies: lanes
    // then touch consecutive shared-memory and global addresses instead of one bank.
    float2 *kspec = spec + (size_t)(MODE == 1 ? row % D : row) * spec_stride;
    for (int pf = threadIdx.x; pf < M; pf += blockDim.x) {
        const int f = bitrev(pf, logM);
        if (f > (M >> 1)) continue;   // the pair (f, M-f) is handled by its smaller member
        const int pm = bitrev((M - f) & (M - 1), logM);
        const float2 Cf = s[phys(pf)], Cm = s[phys(pm)];
        const float2 E = make_float2(0.5f * (Cf.x + Cm.x), 0.5f * (Cf.y - Cm.y));
        const float2 O = make_float2(0.5f * (Cf.y + Cm.y), -0.5f * (Cf.x - Cm.x));
        const float2 wf = tw(f);
        const float2 wO = cmul(wf, O);
        float2 Xf = cadd(E, wO), Xm = cconj(csub(E, wO));
        if (MODE == 0) {
            if (f == 0) {
                kspec[0] = make_float2(E.x + O.x, 0.f);
                kspec[M] = make_float2(E.x - O.x, 0.f);
            } else {
                kspec[pf] = Xf;
                kspec[pm] = Xm;
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
                Yf = cmul(Xf, kspec[pf]);
                Ym = cmul(Xm, kspec[pm]);
            }
            const float2 Ep = make_float2(0.5f * (Yf.x + Ym.x), 0.5f * (Yf.y - Ym.y));
            const float2 Dp = make_float2(0.5f * (Yf.x - Ym.x), 0.5f * (Yf.y + Ym.y));
            const float2 Op = cmulc(Dp, wf);
            s[phys(pf)] = make_float2(Ep.x - Op.y, Ep.y + Op.x);          // E' + i O'
            if (pm != pf) s[phys(pm)] = make_float2(Ep.x + Op.y, -Ep.y + Op.x);  // conj(E') + i conj(O')
        }
    }
    if (MODE == 0) return;
    __syncthreads();
    fft_inverse_dit(s, tw, M, logM);
    const float inv = 1.0f / (float)M;
    for (int n = threadIdx.x; 2 * n < row_stride; n += blockDim.x) {
        const int t = 2 * n;
        float2 p = (n < M) ? s[phys(n)] : make_float2(0.f, 0.f);
        p.x = (t < L) ? p.x * inv : 0.f;
        p.y = (t + 1 < L) ? p.y * inv : 0.f;
        *reinterpret_cast<float2 *>(x + t) = p;
    }
}


// ---- rows longer than one shared-memory FFT: the causal convolution by blocks of kBlockLen tokens (Eq. 6) ----------
//
// With x = (x_0, x_1, ...) and k = (k_0, k_1, ...) cut into blocks of kBlockLen, output block m is
//   y_m = sum_{i+j=m} low(x_i * k_j) + sum_{i+j=m-1} high(x_i * k_j),
// low/high = the two halves of the 2 kBlockLen-point linear convolution of two blocks.  Moving the high half onto the
// low half is a rotation by half a period, i.e. a factor (-1)^f on the spectrum, so one inverse transform per output
// block suffices:  y_m = low( IFFT( sum_{i+j=m} X_i K_j + (-1)^f sum_{i+j=m-1} X_i K_j ) ).
// Block spectra go through global memory in the layout of fft_conv_kernel's mode 0 (M + 1 entries per block: position
// p holds frequency bitrev(p), entry M the Nyquist term).
constexpr int kBlockLen = 16384, kBlockM = 16384, kBlockLogM = 14;

// spectrum of block j = blockIdx.y of row blockIdx.x; rows[row * row_stride + t], t < L
__global__ void __launch_bounds__(1024) fft_block_spectrum_kernel(const float *__restrict__ rows, size_t row_stride, int L, int nb,
                                                                  const float2 *__restrict__ tw_global, float2 *__restrict__ spec)
{
    constexpr int M = kBlockM, logM = kBlockLogM;
    extern __shared__ __align__(16) float2 s[];
    float2 *t1 = s + M, *t2 = t1 + 128;
    for (int j = threadIdx.x; j < 128; j += blockDim.x) {
        t1[j] = tw_global[j];
        t2[j] = tw_global[128 * j];
    }
    const Twiddles tw = {t1, t2};
    const int j = blockIdx.y;
    const size_t row = blockIdx.x;
    const float *x = rows + row * row_stride + (size_t)j * kBlockLen;
    const int len = min(kBlockLen, L - j * kBlockLen);
    for (int n = threadIdx.x; n < M; n += blockDim.x) {
        const int t = 2 * n;
        s[phys(n)] = make_float2(t < len ? x[t] : 0.f, t + 1 < len ? x[t + 1] : 0.f);
    }
    __syncthreads();
    fft_forward_dif(s, tw, M, logM);
    float2 *out = spec + (row * nb + j) * (size_t)(M + 2);
    for (int pf = threadIdx.x; pf < M; pf += blockDim.x) {
        const int f = bitrev(pf, logM);
        if (f > (M >> 1)) continue;
        const int pm = bitrev((M - f) & (M - 1), logM);
        const float2 Cf = s[phys(pf)], Cm = s[phys(pm)];
        const float2 E = make_float2(0.5f * (Cf.x + Cm.x), 0.5f * (Cf.y - Cm.y));
        const float2 O = make_float2(0.5f * (Cf.y + Cm.y), -0.5f * (Cf.x - Cm.x));
        const float2 wO = cmul(tw(f), O);
        if (f == 0) {
            out[0] = make_float2(E.x + O.x, 0.f);
            out[M] = make_float2(E.x - O.x, 0.f);
        } else {
            out[pf] = cadd(E, wO);
            out[pm] = cconj(csub(E, wO));
        }
    }
}

// output block m = blockIdx.y of row blockIdx.x, written over rows[row * row_stride + m * kBlockLen ...]
__global__ void __launch_bounds__(1024) fft_block_combine_kernel(float *__restrict__ rows, size_t row_stride, int L, int D, int nb,
                                                                 const float2 *__restrict__ tw_global,
                                                                 const float2 *__restrict__ xspec, const float2 *__restrict__ kspec)
{
    constexpr int M = kBlockM, logM = kBlockLogM;
    extern __shared__ __align__(16) float2 s[];
    float2 *t1 = s + M, *t2 = t1 + 128;
    for (int j = threadIdx.x; j < 128; j += blockDim.x) {
        t1[j] = tw_global[j];
        t2[j] = tw_global[128 * j];
    }
    __syncthreads();
    const Twiddles tw = {t1, t2};
    const int m = blockIdx.y;
    const size_t row = blockIdx.x;
    const size_t stride = (size_t)(M + 2);
    const float2 *X = xspec + row * nb * stride, *K = kspec + (row % D) * nb * stride;
    for (int pf = threadIdx.x; pf < M; pf += blockDim.x) {
        const int f = bitrev(pf, logM);
        if (f > (M >> 1)) continue;
        const int pm = bitrev((M - f) & (M - 1), logM);
        const float sgn = (f & 1) ? -1.f : 1.f;   // M - f has the parity of f
        float2 Yf = make_float2(0.f, 0.f), Ym = make_float2(0.f, 0.f);
        if (f == 0) {   // entries 0 (DC) and M (Nyquist), both real and of even frequency
            for (int i = 0; i <= m; ++i) {
                Yf.x += X[i * stride].x * K[(m - i) * stride].x;
                Ym.x += X[i * stride + M].x * K[(m - i) * stride + M].x;
            }
            for (int i = 0; i < m; ++i) {
                Yf.x += X[i * stride].x * K[(m - 1 - i) * stride].x;
                Ym.x += X[i * stride + M].x * K[(m - 1 - i) * stride + M].x;
            }
        } else {
            for (int i = 0; i <= m; ++i) {
                Yf = cadd(Yf, cmul(X[i * stride + pf], K[(m - i) * stride + pf]));
                Ym = cadd(Ym, cmul(X[i * stride + pm], K[(m - i) * stride + pm]));
            }
            float2 Hf = make_float2(0.f, 0.f), Hm = make_float2(0.f, 0.f);
            for (int i = 0; i < m; ++i) {
                Hf = cadd(Hf, cmul(X[i * stride + pf], K[(m - 1 - i) * stride + pf]));
                Hm = cadd(Hm, cmul(X[i * stride + pm], K[(m - 1 - i) * stride + pm]));
            }
            Yf = make_float2(Yf.x + sgn * Hf.x, Yf.y + sgn * Hf.y);
            Ym = make_float2(Ym.x + sgn * Hm.x, Ym.y + sgn * Hm.y);
        }
        // packed spectrum of the real result, as in fft_conv_kernel's mode 1
        const float2 wf = tw(f);
        const float2 Ep = make_float2(0.5f * (Yf.x + Ym.x), 0.5f * (Yf.y - Ym.y));
        const float2 Dp = make_float2(0.5f * (Yf.x - Ym.x), 0.5f * (Yf.y + Ym.y));
        const float2 Op = cmulc(Dp, wf);
        s[phys(pf)] = make_float2(Ep.x - Op.y, Ep.y + Op.x);
        if (pm != pf) s[phys(pm)] = make_float2(Ep.x + Op.y, -Ep.y + Op.x);
    }
    __syncthreads();
    fft_inverse_dit(s, tw, M, logM);
    const float inv = 1.0f / (float)M;
    float *y = rows + row * row_stride + (size_t)m * kBlockLen;
    const int len = min(kBlockLen, L - m * kBlockLen);
    for (int n = threadIdx.x; 2 * n < len; n += blockDim.x) {
        const float2 p = s[phys(n)];
        y[2 * n] = p.x * inv;
        if (2 * n + 1 < len) y[2 * n + 1] = p.y * inv;
    }
}

}  // namespace

namespace {
template <typename T>
chela_status_t launch_shortconv_t(const void *x, const float *w, const float *bias, void *y, int B, int L, int D, int width,
                                  int act, cudaStream_t stream)
{
    const int threads = 256, max_blocks = 148 * 32;
    if (width <= 4) {
        constexpr int CH = 4;
        const size_t total = (size_t)B * ((L + 31) / 32) * (D / CH);
        const int blocks = (int)((total + threads - 1) / threads < (size_t)max_blocks ? (total + threads - 1) / threads : max_blocks);
        const T *xi = (const T *)x;
        T *yo = (T *)y;
        switch (width) {
            case 1: shortconv_fast_kernel<T, 1, CH><<<blocks, threads, 0, stream>>>(xi, w, bias, yo, B, L, D, act); break;
            case 2: shortconv_fast_kernel<T, 2, CH><<<blocks, threads, 0, stream>>>(xi, w, bias, yo, B, L, D, act); break;
            case 3: shortconv_fast_kernel<T, 3, CH><<<blocks, threads, 0, stream>>>(xi, w, bias, yo, B, L, D, act); break;
            default: shortconv_fast_kernel<T, 4, CH><<<blocks, threads, 0, stream>>>(xi, w, bias, yo, B, L, D, act); break;
        }
    } else {
        const size_t nvec = (size_t)B * L * (D / 8);
        const int blocks = (int)((nvec + threads - 1) / threads < (size_t)max_blocks * 2 ? (nvec + threads - 1) / threads : max_blocks * 2);
        shortconv_kernel<T><<<blocks, threads, 0, stream>>>((const T *)x, w, bias, (T *)y, B, L, D, width, act);
    }
    return last_launch_status();
}
}  // namespace

chela_status_t launch_shortconv(const void *x, const float *w, const float *bias, void *y, int B, int L,
                                int D, int width, int act, chela_dtype_t io_dtype, cudaStream_t stream)
{
    if (io_dtype == CHELA_BF16) return launch_shortconv_t<__nv_bfloat16>(x, w, bias, y, B, L, D, width, act, stream);
    return launch_shortconv_t<float>(x, w, bias, y, B, L, D, width, act, stream);
}

namespace {
__global__ void reparam_kernel(const float *__restrict__ w1, int width1, const float *__restrict__ w2, int width2,
                               float *__restrict__ merged, int D)
{
    const int wm = max(width1, width2);
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= D * wm) return;
    const int c = i / wm, j = i % wm;
    merged[i] = (j < width1 ? w1[c * width1 + j] : 0.f) + (j < width2 ? w2[c * width2 + j] : 0.f);
}
}  // namespace

chela_status_t launch_shortconv_reparam(const float *w1, int width1, const float *w2, int width2, float *merged, int D,
                                        cudaStream_t stream)
{
    const int n = D * (width1 > width2 ? width1 : width2);
    reparam_kernel<<<(n + 255) / 256, 256, 0, stream>>>(w1, width1, w2, width2, merged, D);
    return last_launch_status();
}

namespace {
struct LongconvPlan {
    int M, logM, Ls, nb;   // nb > 1: the blocked path (L > kBlockLen), M = kBlockM points per block
    size_t off_at, off_tw, off_spec, off_xspec, total;
};
LongconvPlan longconv_plan(int B, int L, int D)
{
    LongconvPlan p;
    p.nb = (L + kBlockLen - 1) / kBlockLen;
    if (p.nb < 1) p.nb = 1;
    p.M = p.nb > 1 ? kBlockM : (next_pow2(L) < 16 ? 16 : next_pow2(L));
    p.logM = 0;
    while ((1 << p.logM) < p.M) ++p.logM;
    p.Ls = (int)align_up((size_t)L, 8);
    p.off_at = 0;
    p.off_tw = align_up(p.off_at + (size_t)B * D * p.Ls * sizeof(float), 256);
    p.off_spec = align_up(p.off_tw + (size_t)p.M * sizeof(float2), 256);
    // kernel spectra: rows of M + 1 entries, 16-byte aligned, one per (channel, block)
    p.off_xspec = align_up(p.off_spec + (size_t)D * p.nb * (p.M + 2) * sizeof(float2), 256);
    // blocked path only: the spectra of the data blocks
    p.total = p.nb > 1 ? align_up(p.off_xspec + (size_t)B * D * p.nb * (p.M + 2) * sizeof(float2), 256) : p.off_xspec;
    return p;
}
const size_t kBlockSmem = (size_t)(kBlockM + 256) * sizeof(float2);
chela_status_t block_kernels_ready()
{
    if (cudaFuncSetAttribute(fft_block_spectrum_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBlockSmem) != cudaSuccess ||
        cudaFuncSetAttribute(fft_block_combine_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBlockSmem) != cudaSuccess)
        return CHELA_ERR_CUDA;
    return CHELA_OK;
}
}  // namespace

size_t longconv_workspace_bytes(int B, int L, int D) { return longconv_plan(B, L, D).total; }
// twiddle table followed by the kernel spectra, as launch_longconv_prepare writes them
static size_t spectrum_off_spec(int L) { return align_up((size_t)longconv_plan(1, L, 1).M * sizeof(float2), 256); }
size_t longconv_spectrum_bytes(int L, int D)
{
    const LongconvPlan p = longconv_plan(1, L, D);
    return align_up(spectrum_off_spec(L) + (size_t)D * p.nb * (p.M + 2) * sizeof(float2), 256);
}
int longconv_row_stride(int L) { return (int)align_up((size_t)L, 8); }
// the FFT kernels that can write bf16 pair rows cover 2^10 .. 2^14 points
bool longconv_transposed_pair_supported(int L) { return L > 512 && L <= 16384; }

// rows [B*D][Ls] back to token-major [B, L, D] in the output dtype
static chela_status_t finish_longconv(const float *at, void *z, int B, int L, int D, int Ls, chela_dtype_t out_dtype,
                                      cudaStream_t stream)
{
    dim3 g2((L + 31) / 32, (D + 63) / 64, B);
    if (out_dtype == CHELA_BF16 || out_dtype == CHELA_BF16_PAIR) {
        dim3 gf((L + 63) / 64, (D + 63) / 64, B);
        transpose_out_bf16_kernel<<<gf, 256, 0, stream>>>(at, (__nv_bfloat16 *)z, L, D, Ls,
                                                          out_dtype == CHELA_BF16_PAIR ? (size_t)B * L * D : 0);
    } else
        transpose_out_kernel<float><<<g2, 256, 0, stream>>>(at, (float *)z, L, D, Ls, 0);
    return last_launch_status();
}

// The part of the long convolution that depends on the weights only (Eq. 6: the spectrum of each zero-padded kernel)
// and the twiddle table, into a caller-owned buffer of longconv_spectrum_bytes(L, D).
chela_status_t launch_longconv_prepare(const float *k_long, int L, int D, void *spectrum, cudaStream_t stream)
{
    const LongconvPlan p = longconv_plan(1, L, D);
    float2 *tw = (float2 *)spectrum;
    float2 *spec = (float2 *)((char *)spectrum + spectrum_off_spec(L));
    twiddle_kernel<<<(p.M + 255) / 256, 256, 0, stream>>>(tw, p.M);
    if (p.nb > 1) {
        if (block_kernels_ready() != CHELA_OK) return CHELA_ERR_CUDA;
        fft_block_spectrum_kernel<<<dim3(D, p.nb), 1024, kBlockSmem, stream>>>(k_long, (size_t)L, L, p.nb, tw, spec);
        return last_launch_status();
    }
    const int spec_stride = p.M + 2;
    if (launch_fft_conv_fast(0, const_cast<float *>(k_long), L, L, D, D, p.logM, tw, spec, spec_stride, stream)) return last_launch_status();
    const size_t smem = (size_t)(p.M + 256) * sizeof(float2);
    int threads = p.M / 16;
    threads = threads < 32 ? 32 : (threads > 1024 ? 1024 : threads);
    if (cudaFuncSetAttribute(fft_conv_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return CHELA_ERR_CUDA;
    fft_conv_kernel<0><<<D, threads, smem, stream>>>(const_cast<float *>(k_long), L, L, D, p.M, p.logM, tw, spec, spec_stride);
    return last_launch_status();
}

chela_status_t launch_longconv(const void *x, const float *k_long, const float *w_short, int short_width,
                               void *z, int B, int L, int D, chela_dtype_t in_dtype,
                               chela_dtype_t out_dtype, void *workspace, cudaStream_t stream, bool transposed_pair,
                               const void *spectrum)
{
    // spectrum: what launch_longconv_prepare wrote for these weights (k_long is then not read), else null
    // transposed_pair: z receives the rows as they leave the FFT kernel, [2][B][D][Ls] bf16 (hi plane, lo plane),
    // and the transpose back to token-major is skipped (the projections read this layout as a transposed operand)
    if (transposed_pair && !longconv_transposed_pair_supported(L)) return CHELA_ERR_UNSUPPORTED;
    const LongconvPlan p = longconv_plan(B, L, D);
    char *ws = (char *)workspace;
    float *at = (float *)(ws + p.off_at);
    float2 *tw = spectrum ? (float2 *)spectrum : (float2 *)(ws + p.off_tw);
    float2 *spec = spectrum ? (float2 *)((char *)spectrum + spectrum_off_spec(L)) : (float2 *)(ws + p.off_spec);

    dim3 g1((L + 63) / 64, (D + 31) / 32, B);
    const int wfast = w_short ? short_width : 0;
    if (in_dtype == CHELA_BF16 && wfast <= 4) {
        dim3 gf((L + 63) / 64, (D + 63) / 64, B);
        const __nv_bfloat16 *xb = (const __nv_bfloat16 *)x;
        switch (wfast) {
            case 0: conv_transpose_bf16_kernel<0><<<gf, 256, 0, stream>>>(xb, w_short, at, L, D, p.Ls); break;
            case 1: conv_transpose_bf16_kernel<1><<<gf, 256, 0, stream>>>(xb, w_short, at, L, D, p.Ls); break;
            case 2: conv_transpose_bf16_kernel<2><<<gf, 256, 0, stream>>>(xb, w_short, at, L, D, p.Ls); break;
            case 3: conv_transpose_bf16_kernel<3><<<gf, 256, 0, stream>>>(xb, w_short, at, L, D, p.Ls); break;
            default: conv_transpose_bf16_kernel<4><<<gf, 256, 0, stream>>>(xb, w_short, at, L, D, p.Ls); break;
        }
    } else if (in_dtype == CHELA_BF16)
        conv_transpose_kernel<__nv_bfloat16><<<g1, 256, 0, stream>>>((const __nv_bfloat16 *)x, w_short, short_width,
                                                                     at, L, D, p.Ls);
    else
        conv_transpose_kernel<float><<<g1, 256, 0, stream>>>((const float *)x, w_short, short_width, at, L, D, p.Ls);
    if (!spectrum) twiddle_kernel<<<(p.M + 255) / 256, 256, 0, stream>>>(tw, p.M);

    if (p.nb > 1) {   // longer than one shared-memory row: block spectra through global memory
        if (transposed_pair) return CHELA_ERR_UNSUPPORTED;
        if (block_kernels_ready() != CHELA_OK) return CHELA_ERR_CUDA;
        float2 *xspec = (float2 *)(ws + p.off_xspec);
        if (!spectrum) fft_block_spectrum_kernel<<<dim3(D, p.nb), 1024, kBlockSmem, stream>>>(k_long, (size_t)L, L, p.nb, tw, spec);
        fft_block_spectrum_kernel<<<dim3(B * D, p.nb), 1024, kBlockSmem, stream>>>(at, (size_t)p.Ls, L, p.nb, tw, xspec);
        fft_block_combine_kernel<<<dim3(B * D, p.nb), 1024, kBlockSmem, stream>>>(at, (size_t)p.Ls, L, D, p.nb, tw, xspec, spec);
        return finish_longconv(at, z, B, L, D, p.Ls, out_dtype, stream);
    }
    // sizes 2^10 .. 2^14: the kernels with compile-time strides; other sizes: the generic kernel below
    const int spec_stride = p.M + 2;
    if ((spectrum || launch_fft_conv_fast(0, const_cast<float *>(k_long), L, L, D, D, p.logM, tw, spec, spec_stride, stream)) &&
        launch_fft_conv_fast(1, at, p.Ls, L, D, B * D, p.logM, tw, spec, spec_stride, stream,
                             transposed_pair ? (__nv_bfloat16 *)z : nullptr, (size_t)B * D * p.Ls)) {
        if (transposed_pair) return last_launch_status();
        return finish_longconv(at, z, B, L, D, p.Ls, out_dtype, stream);
    }
    if (transposed_pair) return CHELA_ERR_UNSUPPORTED;
    const size_t smem = (size_t)(p.M + 256) * sizeof(float2);
    int threads = p.M / 16;
    threads = threads < 32 ? 32 : (threads > 1024 ? 1024 : threads);
    cudaError_t e = cudaFuncSetAttribute(fft_conv_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(fft_conv_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return CHELA_ERR_CUDA;
    if (!spectrum) fft_conv_kernel<0><<<D, threads, smem, stream>>>(const_cast<float *>(k_long), L, L, D, p.M, p.logM, tw, spec, spec_stride);
    fft_conv_kernel<1><<<B * D, threads, smem, stream>>>(at, p.Ls, L, D, p.M, p.logM, tw, spec, spec_stride);
    return finish_longconv(at, z, B, L, D, p.Ls, out_dtype, stream);
}

}  // namespace chela
