// FFT long convolution (Eq. 6, evaluated as a causal linear convolution), sizes 2^10 .. 2^14 complex points.
//
// One CTA per row.  The real row of length <= M is zero-padded to 2M reals and packed into M complex points;
// the M-point transform runs in shared memory as decimation-in-frequency passes (natural order in,
// bit-reversed order out), the spectrum is multiplied with the kernel's in that bit-reversed order, and the
// inverse runs as the mirrored decimation-in-time passes, so no reordering pass exists.
//
// Every thread owns 16 points per pass.  All strides are compile-time constants, so a pass costs one address
// computation per thread and the rest are immediate offsets:
//   first pass    radix 2^R0 (R0 = 1..4) on 16 / 2^R0 groups per thread, reading the packed row from global
//                 memory (forward) or writing the result row to it (inverse);
//   middle passes radix 16 at sub-length 4096 and 256;
//   last pass     radix 16 on 16 contiguous points (128-bit accesses).
// A radix-16 step is a fixed 16-point network (constant roots only) followed by 15 twiddles w^m that are
// powers of one table entry w.
//
// Layout: point e sits at float2 index e + 2 (e >> 4): 16 bytes of padding after every 128 bytes keep the
// contiguous pass free of bank conflicts, and any stride that is a multiple of 16 points stays linear.
#include "common.cuh"

namespace chela {
namespace {

__device__ __forceinline__ float2 cmul(float2 a, float2 b) { return make_float2(a.x * b.x - a.y * b.y, a.x * b.y + a.y * b.x); }
__device__ __forceinline__ float2 cmulc(float2 a, float2 b) { return make_float2(a.x * b.x + a.y * b.y, a.y * b.x - a.x * b.y); }  // a conj(b)
__device__ __forceinline__ float2 csq(float2 a) { return make_float2(a.x * a.x - a.y * a.y, 2.f * a.x * a.y); }
__device__ __forceinline__ float2 cadd(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ float2 csub(float2 a, float2 b) { return make_float2(a.x - b.x, a.y - b.y); }
template <bool kConj>
__device__ __forceinline__ float2 twmul(float2 v, float2 w) { return kConj ? cmulc(v, w) : cmul(v, w); }

// a * exp(-2 pi i n / 16); n is a compile-time constant wherever this is called (unrolled loops)
__device__ __forceinline__ float2 mul_w16(float2 a, int n)
{
    constexpr float c1 = 0.92387953251128674f, s1 = 0.38268343236508977f, h = 0.70710678118654752f;
    switch (n & 15) {
        case 0: return a;
        case 1: return make_float2(a.x * c1 + a.y * s1, a.y * c1 - a.x * s1);
        case 2: return make_float2(h * (a.x + a.y), h * (a.y - a.x));
        case 3: return make_float2(a.x * s1 + a.y * c1, a.y * s1 - a.x * c1);
        case 4: return make_float2(a.y, -a.x);
        case 5: return make_float2(a.y * c1 - a.x * s1, -a.y * s1 - a.x * c1);
        case 6: return make_float2(h * (a.y - a.x), -h * (a.x + a.y));
        case 7: return make_float2(a.y * s1 - a.x * c1, -a.y * c1 - a.x * s1);
        case 8: return make_float2(-a.x, -a.y);
        case 9: return make_float2(-a.x * c1 - a.y * s1, a.x * s1 - a.y * c1);
        case 10: return make_float2(-h * (a.x + a.y), h * (a.x - a.y));
        case 11: return make_float2(-a.x * s1 - a.y * c1, a.x * c1 - a.y * s1);
        case 12: return make_float2(-a.y, a.x);
        case 13: return make_float2(a.x * s1 - a.y * c1, a.y * s1 + a.x * c1);
        case 14: return make_float2(h * (a.x - a.y), h * (a.x + a.y));
        default: return make_float2(a.x * c1 - a.y * s1, a.y * c1 + a.x * s1);
    }
}

__host__ __device__ constexpr int rev_bits(int r, int bits)
{
    int o = 0;
    for (int i = 0; i < bits; ++i) o |= ((r >> i) & 1) << (bits - 1 - i);
    return o;
}

// 2^R-point decimation-in-frequency network on v[base .. base + 2^R): constant roots only; the output of
// frequency digit m ends in register base + rev(m).
template <int R>
__device__ __forceinline__ void dif_net(float2 (&v)[16], int base)
{
    constexpr int G = 1 << R;
#pragma unroll
    for (int st = 0; st < R; ++st) {
        const int h = G >> (st + 1);
#pragma unroll
        for (int blk = 0; blk < (1 << st); ++blk)
#pragma unroll
            for (int jj = 0; jj < h; ++jj) {
                const int ia = base + blk * 2 * h + jj, ib = ia + h;
                const float2 a = v[ia], b = v[ib];
                v[ia] = cadd(a, b);
                v[ib] = mul_w16(csub(a, b), jj * (8 / h));
            }
    }
}
// Its inverse up to the factor 2^R (stages in the opposite order, conjugate roots).
template <int R>
__device__ __forceinline__ void dit_net(float2 (&v)[16], int base)
{
    constexpr int G = 1 << R;
#pragma unroll
    for (int st = R - 1; st >= 0; --st) {
        const int h = G >> (st + 1);
#pragma unroll
        for (int blk = 0; blk < (1 << st); ++blk)
#pragma unroll
            for (int jj = 0; jj < h; ++jj) {
                const int ia = base + blk * 2 * h + jj, ib = ia + h;
                const float2 a = v[ia], bt = mul_w16(v[ib], 16 - jj * (8 / h));
                v[ia] = cadd(a, bt);
                v[ib] = csub(a, bt);
            }
    }
}

// v[rev4(m)] *= w^m (kConj: conj(w)^m), m = 1..15, from w alone: 5 squarings/products give w^2, w^3, w^4,
// w^8, w^12 and every other power is one product of those (at most five roundings deep).
template <bool kConj>
__device__ __forceinline__ void apply_powers16(float2 (&v)[16], float2 b1)
{
    const float2 b2 = csq(b1), b3 = cmul(b2, b1);
    v[8] = twmul<kConj>(v[8], b1);     // m = 1
    v[4] = twmul<kConj>(v[4], b2);     // m = 2
    v[12] = twmul<kConj>(v[12], b3);   // m = 3
    const float2 w4 = csq(b2);
    v[2] = twmul<kConj>(v[2], w4);                  // m = 4
    v[10] = twmul<kConj>(v[10], cmul(w4, b1));      // m = 5
    v[6] = twmul<kConj>(v[6], cmul(w4, b2));        // m = 6
    v[14] = twmul<kConj>(v[14], cmul(w4, b3));      // m = 7
    const float2 w8 = csq(w4);
    v[1] = twmul<kConj>(v[1], w8);                  // m = 8
    v[9] = twmul<kConj>(v[9], cmul(w8, b1));        // m = 9
    v[5] = twmul<kConj>(v[5], cmul(w8, b2));        // m = 10
    v[13] = twmul<kConj>(v[13], cmul(w8, b3));      // m = 11
    const float2 w12 = cmul(w8, w4);
    v[3] = twmul<kConj>(v[3], w12);                 // m = 12
    v[11] = twmul<kConj>(v[11], cmul(w12, b1));     // m = 13
    v[7] = twmul<kConj>(v[7], cmul(w12, b2));       // m = 14
    v[15] = twmul<kConj>(v[15], cmul(w12, b3));     // m = 15
}

__device__ __forceinline__ int pad(int e) { return e + ((e >> 4) << 1); }

// Shared-memory tables, all cut from E(j) = exp(-2 pi i j / 2M), j < M (E(j + M) = -E(j)):
//   t1[j] = E(j), j < 128; t2[j] = E(128 j): E(f) = t1[f & 127] t2[f >> 7] for the real-transform split
//   ta[g] = exp(-2 pi i g / M), g < M/16                (first pass)
//   tb[k] = exp(-2 pi i k / 4096), k < 256              (pass at sub-length 4096)
//   tc[(m-1) * 16 + k] = exp(-2 pi i k m / 256)         (pass at sub-length 256: all 15 powers direct)
struct Tables {
    const float2 *t1, *t2, *ta, *tb, *tc;
};

// ---- passes: slot g (0 <= g < M/16) names the 16 points a thread handles ------------------------------------

// Radix-16 pass at sub-length LEN (4096 or 256), shared memory to shared memory.  Points i0 + j LEN/16 with
// i0 = block * LEN + k.  Forward: network, then point of digit m times W_LEN^(k m).  Inverse: the mirror.
template <int LEN, bool kInverse>
__device__ __forceinline__ void r16_pass(float2 *s, int g, const Tables &tb)
{
    constexpr int q = LEN / 16, PQ = q + q / 8;
    const int k = g & (q - 1);
    const int i0 = ((g - k) << 4) + k;
    float2 *p = s + pad(i0);
    float2 v[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = p[j * PQ];
    if (!kInverse) dif_net<4>(v, 0);
    if (LEN == 256) {
#pragma unroll
        for (int m = 1; m < 16; ++m) v[rev_bits(m, 4)] = twmul<kInverse>(v[rev_bits(m, 4)], tb.tc[(m - 1) * 16 + k]);
    } else {
        apply_powers16<kInverse>(v, tb.tb[k]);
    }
    if (kInverse) dit_net<4>(v, 0);
#pragma unroll
    for (int j = 0; j < 16; ++j) p[j * PQ] = v[j];
}

// Radix-16 pass on the 16 contiguous points of block g: no twiddles outside the network.
template <bool kInverse>
__device__ __forceinline__ void contiguous_pass(float2 *s, int g)
{
    float4 *p = reinterpret_cast<float4 *>(s + 18 * g);
    float2 v[16];
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const float4 t = p[c];
        v[2 * c] = make_float2(t.x, t.y);
        v[2 * c + 1] = make_float2(t.z, t.w);
    }
    if (kInverse) dit_net<4>(v, 0);
    else dif_net<4>(v, 0);
#pragma unroll
    for (int c = 0; c < 8; ++c) p[c] = make_float4(v[2 * c].x, v[2 * c].y, v[2 * c + 1].x, v[2 * c + 1].y);
}

// packed point e of a real row: x[2e] + i x[2e+1], zero past L
__device__ __forceinline__ float2 load_packed(const float *__restrict__ x, int e, int L, bool aligned)
{
    const int t = 2 * e;
    if (t + 1 < L) {
        if (aligned) return *reinterpret_cast<const float2 *>(x + t);
        return make_float2(x[t], x[t + 1]);
    }
    return make_float2(t < L ? x[t] : 0.f, 0.f);
}

// First pass (sub-length M, radix 2^R0) of the forward transform: 16 / 2^R0 groups per thread, group u holds
// points k + j M/2^R0 with k = g + u M/16.  Reads the packed row from global memory.  The twiddle of digit m is
// W_M^(k m) = W_M^(g m) W_16^(u m).
template <int LOGM, int R0>
__device__ __forceinline__ void first_pass_fwd(float2 *s, int g, const Tables &tb, const float *__restrict__ x, int L, bool aligned)
{
    constexpr int M = 1 << LOGM, G0 = 1 << R0, NG = 16 / G0, q0 = M / G0, NT = M / 16;
    constexpr int PQ0 = q0 + q0 / 8, PNT = NT + NT / 8;
    float2 v[16];
#pragma unroll
    for (int u = 0; u < NG; ++u)
#pragma unroll
        for (int j = 0; j < G0; ++j) {
            const int e = g + u * NT + j * q0;
            // the upper half of the packed array is the zero padding
            v[u * G0 + j] = (2 * e < M) ? load_packed(x, e, L, aligned) : make_float2(0.f, 0.f);
        }
#pragma unroll
    for (int u = 0; u < NG; ++u) dif_net<R0>(v, u * G0);
    const float2 b1 = tb.ta[g];
    if (R0 == 4) {
        apply_powers16<false>(v, b1);
    } else {
        float2 pw[8];
        pw[1] = b1;
        if (G0 > 2) { pw[2] = csq(b1); pw[3] = cmul(pw[2], b1); }
        if (G0 > 4) { pw[4] = csq(pw[2]); pw[5] = cmul(pw[4], b1); pw[6] = cmul(pw[4], pw[2]); pw[7] = cmul(pw[4], pw[3]); }
#pragma unroll
        for (int u = 0; u < NG; ++u)
#pragma unroll
            for (int r = 1; r < G0; ++r) {
                const int m = rev_bits(r, R0);
                v[u * G0 + r] = mul_w16(cmul(v[u * G0 + r], pw[m]), u * m);
            }
    }
    float2 *p = s + pad(g);
#pragma unroll
    for (int u = 0; u < NG; ++u)
#pragma unroll
        for (int r = 0; r < G0; ++r) p[u * PNT + r * PQ0] = v[u * G0 + r];
}

// Its mirror, the last pass of the inverse transform: writes the real row (scaled) to global memory; reals
// t >= L are written as zeros up to the row stride.
template <int LOGM, int R0>
__device__ __forceinline__ void first_pass_inv(const float2 *s, int g, const Tables &tb, float *__restrict__ x, int L, int row_stride,
                                               float scale, __nv_bfloat16 *__restrict__ zt_hi, __nv_bfloat16 *__restrict__ zt_lo)
{
    constexpr int M = 1 << LOGM, G0 = 1 << R0, NG = 16 / G0, q0 = M / G0, NT = M / 16;
    constexpr int PQ0 = q0 + q0 / 8, PNT = NT + NT / 8;
    float2 v[16];
    const float2 *p = s + pad(g);
#pragma unroll
    for (int u = 0; u < NG; ++u)
#pragma unroll
        for (int r = 0; r < G0; ++r) v[u * G0 + r] = p[u * PNT + r * PQ0];
    const float2 b1 = tb.ta[g];
    if (R0 == 4) {
        apply_powers16<true>(v, b1);
    } else {
        float2 pw[8];
        pw[1] = b1;
        if (G0 > 2) { pw[2] = csq(b1); pw[3] = cmul(pw[2], b1); }
        if (G0 > 4) { pw[4] = csq(pw[2]); pw[5] = cmul(pw[4], b1); pw[6] = cmul(pw[4], pw[2]); pw[7] = cmul(pw[4], pw[3]); }
#pragma unroll
        for (int u = 0; u < NG; ++u)
#pragma unroll
            for (int r = 1; r < G0; ++r) {
                const int m = rev_bits(r, R0);
                v[u * G0 + r] = mul_w16(cmulc(v[u * G0 + r], pw[m]), 16 - ((u * m) & 15));
            }
    }
#pragma unroll
    for (int u = 0; u < NG; ++u) dit_net<R0>(v, u * G0);
#pragma unroll
    for (int u = 0; u < NG; ++u)
#pragma unroll
        for (int j = 0; j < G0; ++j) {
            const int t = 2 * (g + u * NT + j * q0);
            if (t < row_stride) {   // row_stride is even
                const float2 o = v[u * G0 + j];
                const float r0 = t < L ? o.x * scale : 0.f, r1 = t + 1 < L ? o.y * scale : 0.f;
                if (zt_hi) {   // bf16 pair rows (hi plane, lo plane) instead of the fp32 row
                    const __nv_bfloat162 hh = __floats2bfloat162_rn(r0, r1);
                    const float2 hf = __bfloat1622float2(hh);
                    *reinterpret_cast<__nv_bfloat162 *>(zt_hi + t) = hh;
                    *reinterpret_cast<__nv_bfloat162 *>(zt_lo + t) = __floats2bfloat162_rn(r0 - hf.x, r1 - hf.y);
                } else {
                    *reinterpret_cast<float2 *>(x + t) = make_float2(r0, r1);
                }
            }
        }
}

// ---- spectrum of the real sequence from the packed transform, product with the kernel, and back ----------------
//
// C[f] (packed transform) sits at position bitrev(f).  For the pair (f, M - f), w = E(f):
//   Ev = (C[f] + conj C[M-f]) / 2,  Od = -i (C[f] - conj C[M-f]) / 2,
//   X[f] = Ev + w Od,  X[M-f] = conj(Ev - w Od)                         (spectrum of the 2M real samples)
//   Y = X K;  E' = (Y[f] + conj Y[M-f]) / 2,  O' = (Y[f] - conj Y[M-f]) / 2 conj(w)
//   C'[f] = E' + i O',  C'[M-f] = conj(E') + i conj(O')                  (packed transform of the product)
// The kernel spectrum is stored in the same position order: entry p holds K[bitrev(p)], entry M the Nyquist term.
template <int MODE>
__device__ __forceinline__ void merge_pair(float2 &Cf, float2 &Cm, float2 w, float2 &Kf, float2 &Km)
{
    const float2 Ev = make_float2(0.5f * (Cf.x + Cm.x), 0.5f * (Cf.y - Cm.y));
    const float2 Od = make_float2(0.5f * (Cf.y + Cm.y), -0.5f * (Cf.x - Cm.x));
    const float2 wO = cmul(w, Od);
    const float2 Xf = cadd(Ev, wO), Xm = make_float2(Ev.x - wO.x, wO.y - Ev.y);
    if (MODE == 0) {
        Kf = Xf;
        Km = Xm;
    } else {
        const float2 Yf = cmul(Xf, Kf), Ym = cmul(Xm, Km);
        const float2 Ep = make_float2(0.5f * (Yf.x + Ym.x), 0.5f * (Yf.y - Ym.y));
        const float2 Dp = make_float2(0.5f * (Yf.x - Ym.x), 0.5f * (Yf.y + Ym.y));
        const float2 Op = cmulc(Dp, w);
        Cf = make_float2(Ep.x - Op.y, Ep.y + Op.x);
        Cm = make_float2(Ep.x + Op.y, Op.x - Ep.y);
    }
}

// Quad i (0 <= i < M/4): the 16-byte chunks at positions (4i, 4i+1) and (pb-1, pb), pb = bitrev(M - f),
// f = bitrev(4i) < M/4, hold the two pairs (f, M-f) and (M/2-f, M/2+f).  Quad 0 instead holds f = 0 with the
// Nyquist term, the self-paired f = M/2, and (in chunk 2,3) the pair (M/4, 3M/4).
template <int LOGM, int MODE>
__device__ __forceinline__ void merge_quad(float2 *s, int i, const Tables &tb, float2 *__restrict__ kspec)
{
    constexpr int M = 1 << LOGM;
    const int pa = 4 * i;
    if (i == 0) {
        float4 *ca = reinterpret_cast<float4 *>(s), *kc = reinterpret_cast<float4 *>(kspec);
        float4 a = ca[0], b = ca[1];
        float4 ka = make_float4(0.f, 0.f, 0.f, 0.f), kb = ka;
        float2 knyq = make_float2(0.f, 0.f);
        if (MODE == 1) {
            ka = kc[0];
            kb = kc[1];
            knyq = kspec[M];
        }
        // f = 0: X[0] = Re + Im, X[M] = Re - Im (both real)
        {
            const float x0 = a.x + a.y, xn = a.x - a.y;
            if (MODE == 0) {
                ka.x = x0; ka.y = 0.f;
                knyq = make_float2(xn, 0.f);
            } else {
                const float y0 = x0 * ka.x, yn = xn * knyq.x;
                a.x = 0.5f * (y0 + yn);
                a.y = 0.5f * (y0 - yn);
            }
        }
        // f = M/2 (its own partner), w = -i
        {
            float2 Cf = make_float2(a.z, a.w), Cm = Cf, Kf = make_float2(ka.z, ka.w), Km = Kf;
            merge_pair<MODE>(Cf, Cm, make_float2(0.f, -1.f), Kf, Km);
            if (MODE == 0) { ka.z = Kf.x; ka.w = Kf.y; }
            else { a.z = Cf.x; a.w = Cf.y; }
        }
        // (M/4, 3M/4) at positions 2, 3; w = E(M/4) = exp(-i pi / 4)
        {
            float2 Cf = make_float2(b.x, b.y), Cm = make_float2(b.z, b.w), Kf = make_float2(kb.x, kb.y), Km = make_float2(kb.z, kb.w);
            merge_pair<MODE>(Cf, Cm, make_float2(0.70710678118654752f, -0.70710678118654752f), Kf, Km);
            if (MODE == 0) kb = make_float4(Kf.x, Kf.y, Km.x, Km.y);
            else b = make_float4(Cf.x, Cf.y, Cm.x, Cm.y);
        }
        if (MODE == 0) {
            kc[0] = ka;
            kc[1] = kb;
            kspec[M] = knyq;
        } else {
            ca[0] = a;
            ca[1] = b;
        }
        return;
    }
    const int f = (int)(__brev((unsigned)pa) >> (32 - LOGM));
    const int pb = (int)(__brev((unsigned)(M - f)) >> (32 - LOGM));   // odd; pb - 1 holds M/2 - f
    float4 *ca = reinterpret_cast<float4 *>(s + pad(pa)), *cb = reinterpret_cast<float4 *>(s + pad(pb - 1));
    float4 *kca = reinterpret_cast<float4 *>(kspec + pa), *kcb = reinterpret_cast<float4 *>(kspec + pb - 1);
    float4 a = ca[0], b = cb[0];
    float4 ka = make_float4(0.f, 0.f, 0.f, 0.f), kb = ka;
    if (MODE == 1) {
        ka = *kca;
        kb = *kcb;
    }
    const float2 w = cmul(tb.t1[f & 127], tb.t2[f >> 7]);
    // pair (f, M - f): positions pa and pb
    float2 Cf = make_float2(a.x, a.y), Cm = make_float2(b.z, b.w), Kf = make_float2(ka.x, ka.y), Km = make_float2(kb.z, kb.w);
    merge_pair<MODE>(Cf, Cm, w, Kf, Km);
    // pair (M/2 - f, M/2 + f): positions pb - 1 and pa + 1; E(M/2 - f) = -i conj(E(f))
    float2 Cf2 = make_float2(b.x, b.y), Cm2 = make_float2(a.z, a.w), Kf2 = make_float2(kb.x, kb.y), Km2 = make_float2(ka.z, ka.w);
    merge_pair<MODE>(Cf2, Cm2, make_float2(-w.y, -w.x), Kf2, Km2);
    if (MODE == 0) {
        *kca = make_float4(Kf.x, Kf.y, Km2.x, Km2.y);
        *kcb = make_float4(Kf2.x, Kf2.y, Km.x, Km.y);
    } else {
        ca[0] = make_float4(Cf.x, Cf.y, Cm2.x, Cm2.y);
        cb[0] = make_float4(Cf2.x, Cf2.y, Cm.x, Cm.y);
    }
}

// MODE 0: rows = long kernels k[D][L]; writes the spectrum spec[row] (position order, see above).
// MODE 1: rows = sequences [B*D][row_stride]; multiplies with spec[row % D] and writes the causal convolution
//         back over the row.
template <int LOGM, int MODE, int NTHR>
__global__ void __launch_bounds__(NTHR) fft_conv_fast_kernel(float *__restrict__ rows, int row_stride, int L, int D,
                                                             const float2 *__restrict__ tw_global, float2 *__restrict__ spec,
                                                             int spec_stride, __nv_bfloat16 *__restrict__ zt, size_t zt_lo_offset)
{
    constexpr int M = 1 << LOGM, NSLOT = M / 16, R0 = ((LOGM - 1) & 3) + 1, LEN1 = M >> R0;
    static_assert(LEN1 == 4096 || LEN1 == 256, "middle passes cover sub-lengths 4096 and 256");
    static_assert(NSLOT % NTHR == 0, "slots per thread");
    extern __shared__ __align__(16) float2 s[];
    float2 *t1 = s + M + M / 8, *t2 = t1 + 128, *ta = t2 + 128, *tbl = ta + NSLOT, *tc = tbl + 256;
    // E(j) for any j >= 0
    auto E = [&](int j) {
        const float2 e = tw_global[j & (M - 1)];
        return ((j >> LOGM) & 1) ? make_float2(-e.x, -e.y) : e;
    };
    for (int j = threadIdx.x; j < 128; j += NTHR) {
        t1[j] = E(j);
        t2[j] = E(128 * j);   // entries past M / 128 are never read
    }
    for (int j = threadIdx.x; j < NSLOT; j += NTHR) ta[j] = E(2 * j);
    if (M >= 4096)
        for (int j = threadIdx.x; j < 256; j += NTHR) tbl[j] = E(j * (2 * M / 4096));
    for (int j = threadIdx.x; j < 240; j += NTHR) {
        const int m = j / 16 + 1, k = j % 16;
        tc[j] = E(k * m * (2 * M / 256));
    }
    const Tables tb = {t1, t2, ta, tbl, tc};
    const int row = blockIdx.x;
    float *x = rows + (size_t)row * row_stride;
    const bool aligned = (reinterpret_cast<size_t>(x) & 7) == 0;
    float2 *kspec = spec + (size_t)(MODE == 1 ? row % D : row) * spec_stride;
    __syncthreads();
    // With one slot per thread the middle passes do not need the whole CTA to meet: the pass at sub-length 4096 works
    // inside blocks of 4096 points, which belong to groups of 256 consecutive threads before and after it, and the pass
    // at sub-length 256 and the contiguous pass work inside blocks of 256 points = 16 consecutive threads of one warp.
    constexpr bool kOneSlot = NSLOT == NTHR;
    auto sync_4096_group = [&]() {
        if (kOneSlot && NTHR > 256) asm volatile("bar.sync %0, 256;" ::"r"(1 + (int)(threadIdx.x >> 8)) : "memory");
        else __syncthreads();
    };
    auto sync_256_group = [&]() {
        if (kOneSlot) __syncwarp();
        else __syncthreads();
    };

    // ---- forward ----
#pragma unroll 1
    for (int g = threadIdx.x; g < NSLOT; g += NTHR) first_pass_fwd<LOGM, R0>(s, g, tb, x, L, aligned);
    __syncthreads();
    if (LEN1 == 4096) {   // sub-length left by the first pass: 4096 or 256
#pragma unroll 1
        for (int g = threadIdx.x; g < NSLOT; g += NTHR) r16_pass<4096, false>(s, g, tb);
        sync_4096_group();
    }
    if (LEN1 >= 256) {
#pragma unroll 1
        for (int g = threadIdx.x; g < NSLOT; g += NTHR) r16_pass<256, false>(s, g, tb);
        sync_256_group();
    }
#pragma unroll 1
    for (int g = threadIdx.x; g < NSLOT; g += NTHR) contiguous_pass<false>(s, g);
    __syncthreads();

    // ---- spectrum product (or spectrum output) ----
#pragma unroll 1
    for (int i = threadIdx.x; i < M / 4; i += NTHR) merge_quad<LOGM, MODE>(s, i, tb, kspec);
    if (MODE == 0) return;
    __syncthreads();

    // ---- inverse ----
#pragma unroll 1
    for (int g = threadIdx.x; g < NSLOT; g += NTHR) contiguous_pass<true>(s, g);
    if (LEN1 >= 256) {
        sync_256_group();
#pragma unroll 1
        for (int g = threadIdx.x; g < NSLOT; g += NTHR) r16_pass<256, true>(s, g, tb);
        if (LEN1 == 4096) sync_4096_group();
        else __syncthreads();
    } else
        __syncthreads();
    if (LEN1 == 4096) {
#pragma unroll 1
        for (int g = threadIdx.x; g < NSLOT; g += NTHR) r16_pass<4096, true>(s, g, tb);
        __syncthreads();
    }
    const float scale = 1.0f / (float)M;
#pragma unroll 1
    // zt given: the result leaves as bf16 pair rows [row][row_stride] (the layout the projections read as a transposed
    // operand) instead of overwriting the fp32 row
    __nv_bfloat16 *zh = zt ? zt + (size_t)row * row_stride : nullptr;
    for (int g = threadIdx.x; g < NSLOT; g += NTHR) first_pass_inv<LOGM, R0>(s, g, tb, x, L, row_stride, scale, zh, zh + zt_lo_offset);
}

template <int LOGM, int NTHR>
bool launch_fast_t(int mode, float *rows, int row_stride, int L, int D, int nrows, const float2 *tw, float2 *spec, int spec_stride,
                   cudaStream_t stream, __nv_bfloat16 *zt, size_t zt_lo_offset)
{
    constexpr int M = 1 << LOGM;
    const size_t smem = (size_t)(M + M / 8 + 128 + 128 + M / 16 + 256 + 256) * sizeof(float2);
    if (mode == 0) {
        auto kern = fft_conv_fast_kernel<LOGM, 0, NTHR>;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return false;
        kern<<<nrows, NTHR, smem, stream>>>(rows, row_stride, L, D, tw, spec, spec_stride, nullptr, 0);
    } else {
        auto kern = fft_conv_fast_kernel<LOGM, 1, NTHR>;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return false;
        kern<<<nrows, NTHR, smem, stream>>>(rows, row_stride, L, D, tw, spec, spec_stride, zt, zt_lo_offset);
    }
    return true;
}

}  // namespace

// True if the size is covered (2^10 <= M <= 2^14) and the kernel was enqueued.  `tw` holds exp(-2 pi i j / 2M),
// j < M; rows of mode 1 must be 8-byte aligned with an even stride.  zt (mode 1, optional): write the result as bf16
// pair rows [nrows][row_stride] at zt and zt + zt_lo_offset instead of over the fp32 rows.
bool launch_fft_conv_fast(int mode, float *rows, int row_stride, int L, int D, int nrows, int logM, const float2 *tw, float2 *spec,
                          int spec_stride, cudaStream_t stream, __nv_bfloat16 *zt, size_t zt_lo_offset)
{
    if (mode == 1 && (row_stride & 1)) return false;
    switch (logM) {
        case 10: return launch_fast_t<10, 64>(mode, rows, row_stride, L, D, nrows, tw, spec, spec_stride, stream, zt, zt_lo_offset);
        case 11: return launch_fast_t<11, 128>(mode, rows, row_stride, L, D, nrows, tw, spec, spec_stride, stream, zt, zt_lo_offset);
        case 12: return launch_fast_t<12, 256>(mode, rows, row_stride, L, D, nrows, tw, spec, spec_stride, stream, zt, zt_lo_offset);
        case 13: return launch_fast_t<13, 512>(mode, rows, row_stride, L, D, nrows, tw, spec, spec_stride, stream, zt, zt_lo_offset);
#ifndef CHELA_FFT14_THREADS
#define CHELA_FFT14_THREADS 1024
#endif
        case 14: return launch_fast_t<14, CHELA_FFT14_THREADS>(mode, rows, row_stride, L, D, nrows, tw, spec, spec_stride, stream, zt, zt_lo_offset);
        default: return false;
    }
}

}  // namespace chela
