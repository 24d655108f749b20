// Dense projection on the sm_100a tensor cores for the Q/K/V formation of the mixer (Eqs. 10-12 in
// their dense form): Y = act(A W + bias), fp32 accumulation in TMEM.
//
// A [M, K] is bf16, or a bf16 pair (A = A_hi + A_lo, two planes): the long-convolution output and the
// resulting Q, K must keep about 16 mantissa bits, because the normalised attention output loses its
// leading digits to cancellation in Q K^T.  W [K, N] is bf16.  Y [M, N] is written as bf16 or as a
// bf16 pair (hi = round(y), lo = round(y - hi)).
//
// Persistent kernel, one CTA per SM, 128 x BN output tiles (BN = 256 when N allows, else 128), K blocks of 64:
//   warp 4 lane 0 : TMA producer (A_hi, A_lo: [128 rows] x 128 B K-major tiles; W: BN / 64 atoms of
//                   [64 k-rows] x 128 B, MN-major), 3- or 4-stage ring (192 KB in flight at BN = 256)
//   warp 5 lane 0 : tcgen05.mma issuer, M = 128, N = BN (BN / 2 cycles per instruction: full rate);
//                   accumulators double-buffered in TMEM (2 x BN columns)
//   warps 0-3     : epilogue: TMEM -> bias, activation, hi/lo split -> swizzled staging -> TMA store,
//                   32 rows x 64 columns per warp and box (ping-pong staging at BN = 128)
// Every wait is bounded; a timeout records CHELA_ERR_TIMEOUT in the status word and ends the CTA cleanly.
#include "sm100_ptx.cuh"

namespace chela {
namespace {

using namespace sm100;

constexpr int BM = 128, BK = 64;
constexpr int kThreads = 192;
constexpr int kATile = BM * 128;        // 16 KB
constexpr int kMaxStages = 4;

// BN = 256 where N allows: the SM takes its operands from L2 at about 45 bytes per clock, which a 128 x 128
// tile with a pair A operand exceeds; a 128 x 256 tile needs two thirds of the bytes per flop.
template <int BN, bool kAPair>
struct Smem {
    static constexpr int kBTile = BK * 128 * (BN / 64);             // BN / 64 atoms of 64 columns
    static constexpr int kStageBytes = (kAPair ? 2 : 1) * kATile + kBTile;
    static constexpr int kStages = (BN == 256 && !kAPair) ? 4 : 3;  // 192 KB of operands in flight at BN = 256
    static constexpr int kStagingBufs = BN == 256 ? 1 : 2;          // per warp: buffers of (hi, lo) x [32 rows x 128 B]
    static constexpr int kStagingWarp = kStagingBufs * 2 * 32 * 128;
    static constexpr int offStage = 0;
    static constexpr int offStaging = kStages * kStageBytes;
    static constexpr int offBar = offStaging + 4 * kStagingWarp;   // full[kStages], empty[kStages], tfull[2], tempty[2]
    static constexpr int offTmem = offBar + 8 * (2 * kMaxStages + 4);
    static constexpr int offAbort = offTmem + 8;
    static constexpr int bytes = offAbort + 8;
    static_assert(bytes <= 232448, "shared memory per CTA");
};

// One box of the epilogue: 64 accumulator values of a row -> bias, activation ACT, bf16 (hi) and the rounding remainder
// (lo).  The activation is a template argument and the caller branches once per box: with a run-time switch per element
// the box's code is three times as long and the epilogue warps wait for instruction fetches.
template <int ACT, bool kYPair>
__device__ __forceinline__ void pack_box(const float (&acc)[64], const float *__restrict__ bias, uint32_t (&wh)[8][4], uint32_t (&wl)[8][4])
{
#pragma unroll
    for (int j8 = 0; j8 < 8; ++j8) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int col = j8 * 8 + e * 2;
            float x0 = acc[col], x1 = acc[col + 1];
            if (bias) {
                x0 += bias[col];
                x1 += bias[col + 1];
            }
            if (ACT) {
                x0 = activate(x0, ACT);
                x1 = activate(x1, ACT);
            }
            const __nv_bfloat162 hh = __floats2bfloat162_rn(x0, x1);
            wh[j8][e] = *reinterpret_cast<const uint32_t *>(&hh);
            if (kYPair) {
                const float2 hf = __bfloat1622float2(hh);
                wl[j8][e] = pack_bf16(x0 - hf.x, x1 - hf.y);
            }
        }
    }
}

// kATrans: A is given transposed, [B][K][Lt] per plane (the long convolution's row layout: channel-major, tokens
// contiguous); its tiles are then MN-major like W's, two 64-token atoms per 128-row tile, and row tile m0 lies in
// batch m0 / Lt at token m0 % Lt (Lt a multiple of 128).
template <int BN, bool kAPair, bool kYPair, bool kATrans = false>
__global__ void __launch_bounds__(kThreads)
gemm_sm100_kernel(const __grid_constant__ CUtensorMap tm_a_hi, const __grid_constant__ CUtensorMap tm_a_lo,
                  const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_y_hi,
                  const __grid_constant__ CUtensorMap tm_y_lo, const float *__restrict__ bias, int M, int N, int K,
                  int act, int *__restrict__ status, int Lt, const WaitCtl wc)
{
    using Smem = Smem<BN, kAPair>;
    constexpr int kStages = Smem::kStages, kStageBytes = Smem::kStageBytes, kStagingWarp = Smem::kStagingWarp;
    constexpr int kAOff = (kAPair ? 2 : 1) * kATile;   // W atoms follow the A tile(s) of a stage
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    if (sbase & 1023u) {
        if (threadIdx.x == 0) atomicExch(status, (int)CHELA_ERR_CUDA);
        return;
    }
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t bar_full0 = sbase + Smem::offBar, bar_empty0 = bar_full0 + 8 * kStages,
                   bar_tfull0 = bar_empty0 + 8 * kStages, bar_tempty0 = bar_tfull0 + 16;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + Smem::offTmem);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + Smem::offAbort);

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar_full0 + 8 * s, 1);
            mbar_init(bar_empty0 + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_tfull0 + 8 * b, 1);
            mbar_init(bar_tempty0 + 8 * b, 4);
        }
        *abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tm_a_hi);
        tma_prefetch_desc(&tm_w);
        tma_prefetch_desc(&tm_y_hi);
    }
    if (warp == 0) {
        tmem_alloc(sbase + Smem::offTmem, 2 * BN);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    const int n_tiles = N / BN, m_tiles = (M + BM - 1) / BM, tiles = n_tiles * m_tiles, kblocks = K / BK;

    if (warp == 4) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int it = 0, issued = 0;
            bool ok = true;
            for (int t = blockIdx.x; ok && t < tiles; t += gridDim.x) {
                const int m0 = (t / n_tiles) * BM, n0 = (t % n_tiles) * BN;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % kStages;
                    ok = mbar_wait(bar_empty0 + 8 * s, ((it / kStages) & 1) ^ 1, abort_flag, wc.limit);
                    if (!ok) break;
                    const uint32_t bar = bar_full0 + 8 * s, dst = sbase + Smem::offStage + s * kStageBytes;
                    mbar_expect_tx(bar, kStageBytes);
                    if (kATrans) {
                        const int bb = m0 / Lt, t0 = m0 % Lt;
#pragma unroll
                        for (int a = 0; a < 2; ++a) {
                            tma_load_3d(dst + a * (kATile / 2), &tm_a_hi, bar, t0 + 64 * a, kb * BK, bb);
                            if (kAPair) tma_load_3d(dst + kATile + a * (kATile / 2), &tm_a_lo, bar, t0 + 64 * a, kb * BK, bb);
                        }
                    } else {
                        tma_load_2d(dst, &tm_a_hi, bar, kb * BK, m0);
                        if (kAPair) tma_load_2d(dst + kATile, &tm_a_lo, bar, kb * BK, m0);
                    }
#pragma unroll
                    for (int a = 0; a < BN / 64; ++a) tma_load_2d(dst + kAOff + a * BK * 128, &tm_w, bar, n0 + 64 * a, kb * BK);
                    issued = it + 1;
                }
            }
            if (!ok) {
                *abort_flag = 1;
                atomicExch(status, (int)CHELA_ERR_TIMEOUT);
                // loads still in flight land in this CTA's shared memory: wait for them (bounded)
                for (int c = issued > kStages ? issued - kStages : 0; c < issued; ++c) mbar_wait(bar_full0 + 8 * (c % kStages), (c / kStages) & 1, nullptr, wc.limit);
            }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(BM, BN, kATrans ? 1 : 0, 1);
            int it = 0, ti = 0;
            bool ok = true;
            for (int t = blockIdx.x; ok && t < tiles; t += gridDim.x, ++ti) {
                const int buf = ti & 1;
                ok = mbar_wait(bar_tempty0 + 8 * buf, ((ti >> 1) & 1) ^ 1, abort_flag, wc.limit);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d = tmem + buf * BN;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % kStages;
                    ok = mbar_wait(bar_full0 + 8 * s, (it / kStages) & 1, abort_flag, wc.limit);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t st = sbase + Smem::offStage + s * kStageBytes;
                    // K-major A: +32 bytes per K step along the row; MN-major A (kATrans): two atoms, +16 rows per K step
                    const uint32_t a_hi = kATrans ? desc_lo(st, kATile / 2) : desc_lo(st),
                                   a_lo = kATrans ? desc_lo(st + kATile, kATile / 2) : desc_lo(st + kATile),
                                   w_lo = desc_lo(st + kAOff, BK * 128);
                    constexpr uint32_t a_step = kATrans ? 128 : 2;
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k) {
                        umma_bf16(d, a_hi + a_step * k, w_lo + 128 * k, idesc, (kb > 0 || k > 0) ? 1u : 0u);
                        if (kAPair) umma_bf16(d, a_lo + a_step * k, w_lo + 128 * k, idesc, 1u);
                    }
                    umma_commit(bar_empty0 + 8 * s);
                }
                if (ok) umma_commit(bar_tfull0 + 8 * buf);
            }
            if (!ok) {
                *abort_flag = 1;
                atomicExch(status, (int)CHELA_ERR_TIMEOUT);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        // thread = accumulator row (TMEM lane); warp w stores rows 32w..32w+31 of the tile
        uint8_t *stg = smem + Smem::offStaging + warp * kStagingWarp;
        const uint32_t stg_u32 = sbase + Smem::offStaging + warp * kStagingWarp;
        int ti = 0, nbox = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < tiles; t += gridDim.x, ++ti) {
            const int m0 = (t / n_tiles) * BM, n0 = (t % n_tiles) * BN, buf = ti & 1;
            ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull0 + 8 * buf, (ti >> 1) & 1, abort_flag, wc.limit));
            if (!ok) break;
            tc_fence_after();
            const uint32_t trow = tmem + ((uint32_t)(warp * 32) << 16) + buf * BN;
#pragma unroll 1
            for (int c = 0; c < BN / 64; ++c, ++nbox) {
                float acc[64];
                tmem_ld32(trow + c * 64, *reinterpret_cast<float(*)[32]>(&acc[0]));
                tmem_ld32(trow + c * 64 + 32, *reinterpret_cast<float(*)[32]>(&acc[32]));
                tmem_ld_wait();
                if (c == BN / 64 - 1) {
                    // the accumulator is in registers: hand the TMEM buffer back to the issuer
                    tc_fence_before();
                    __syncwarp();
                    // (test hook: the first hand-back of CTA 0 left out, so that the issuer's wait for it runs out)
                    if (lane == 0 && !(wc.skip_arrival && blockIdx.x == 0 && ti == 0 && warp == 0)) mbar_arrive(bar_tempty0 + 8 * buf);
                }
                // bias, activation and the hi/lo split first, into registers: the store of the previous box is still
                // reading the staging buffer meanwhile
                uint32_t wh[8][4], wl[8][4];
                const float *bias_box = bias ? bias + n0 + c * 64 : nullptr;
                if (act == 0) pack_box<0, kYPair>(acc, bias_box, wh, wl);
                else if (act == 1) pack_box<1, kYPair>(acc, bias_box, wh, wl);
                else pack_box<2, kYPair>(acc, bias_box, wh, wl);
                // the staging buffer is free once the store that last used it has been read (two boxes ago with
                // ping-pong buffers, the previous box with one)
                if (lane == 0) {
                    if (Smem::kStagingBufs == 2) bulk_wait_read1();
                    else bulk_wait_read0();
                }
                __syncwarp();
                const int sb = Smem::kStagingBufs == 2 ? (nbox & 1) : 0;
                uint8_t *hi = stg + sb * (2 * 32 * 128), *lo = hi + 32 * 128;
#pragma unroll
                for (int j8 = 0; j8 < 8; ++j8) {
                    const uint32_t off = sw128(lane, j8);
                    *reinterpret_cast<uint4 *>(hi + off) = make_uint4(wh[j8][0], wh[j8][1], wh[j8][2], wh[j8][3]);
                    if (kYPair) *reinterpret_cast<uint4 *>(lo + off) = make_uint4(wl[j8][0], wl[j8][1], wl[j8][2], wl[j8][3]);
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) {   // rows past M are clipped by the copy engine
                    const uint32_t src = stg_u32 + sb * (2 * 32 * 128);
                    tma_store_2d(&tm_y_hi, src, n0 + c * 64, m0 + warp * 32);
                    if (kYPair) tma_store_2d(&tm_y_lo, src + 32 * 128, n0 + c * 64, m0 + warp * 32);
                    bulk_commit();
                }
            }
        }
        if (!ok && lane == 0) {
            *abort_flag = 1;
            atomicExch(status, (int)CHELA_ERR_TIMEOUT);
        }
        if (lane == 0) bulk_wait0();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 2 * BN);
}

bool map_2d(CUtensorMap *map, const void *ptr, size_t rows, int cols, int box_cols, int box_rows)
{
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    return make_map_sw128(map, ptr, false, 2, dims, strides, box);
}

}  // namespace

bool gemm_sm100_supported(size_t M, int K, int N, chela_dtype_t a_dtype, chela_dtype_t w_dtype, chela_dtype_t y_dtype)
{
    return M >= 1 && M < (1ull << 31) && K % BK == 0 && N % 128 == 0 && w_dtype == CHELA_BF16 &&
           (a_dtype == CHELA_BF16 || a_dtype == CHELA_BF16_PAIR) && (y_dtype == CHELA_BF16 || y_dtype == CHELA_BF16_PAIR);
}

// a, y: for a bf16 pair the low plane follows the high plane (M*K resp. M*N elements later).
chela_status_t launch_gemm_sm100(const void *a, const void *w, const float *bias, void *y, size_t M, int K, int N,
                                 int act, chela_dtype_t a_dtype, chela_dtype_t y_dtype, int *status, cudaStream_t stream)
{
    const bool a_pair = a_dtype == CHELA_BF16_PAIR, y_pair = y_dtype == CHELA_BF16_PAIR;
    const __nv_bfloat16 *a_hi = (const __nv_bfloat16 *)a, *a_lo = a_pair ? a_hi + M * K : a_hi;
    __nv_bfloat16 *y_hi = (__nv_bfloat16 *)y, *y_lo = y_pair ? y_hi + M * N : y_hi;
    CUtensorMap ma_hi, ma_lo, mw, my_hi, my_lo;
    if (!map_2d(&ma_hi, a_hi, M, K, BK, BM) || !map_2d(&ma_lo, a_lo, M, K, BK, BM) || !map_2d(&mw, w, K, N, 64, BK) ||
        !map_2d(&my_hi, y_hi, M, N, 64, 32) || !map_2d(&my_lo, y_lo, M, N, 64, 32))
        return CHELA_ERR_CUDA;
    int sms = 0, dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        sms = 148;
    const int bn = (N % 256 == 0) ? 256 : 128;
    const long long tiles = (long long)((M + BM - 1) / BM) * (N / bn);
    const int grid = (int)(tiles < sms ? tiles : sms);
    typedef void (*Kern)(CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, const float *, int, int, int, int, int *, int, WaitCtl);
    Kern kern;
    int smem;
    if (bn == 256) {
        kern = a_pair ? (y_pair ? gemm_sm100_kernel<256, true, true> : gemm_sm100_kernel<256, true, false>)
                      : (y_pair ? gemm_sm100_kernel<256, false, true> : gemm_sm100_kernel<256, false, false>);
        smem = a_pair ? Smem<256, true>::bytes : Smem<256, false>::bytes;
    } else {
        kern = a_pair ? (y_pair ? gemm_sm100_kernel<128, true, true> : gemm_sm100_kernel<128, true, false>)
                      : (y_pair ? gemm_sm100_kernel<128, false, true> : gemm_sm100_kernel<128, false, false>);
        smem = a_pair ? Smem<128, true>::bytes : Smem<128, false>::bytes;
    }
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return CHELA_ERR_CUDA;
    kern<<<grid, kThreads, smem, stream>>>(ma_hi, ma_lo, mw, my_hi, my_lo, bias, (int)M, N, K, act, status, 0, current_wait_ctl());
    return last_launch_status();
}

bool gemm_sm100_at_supported(int B, int L, int Ls, int K, int N)
{
    return B >= 1 && L % BM == 0 && Ls % 8 == 0 && Ls >= L && K % BK == 0 && N % 256 == 0;
}

// Y [B*L, N] = act(A W + bias) with A given transposed as a bf16 pair: at = [2][B][K][Ls] (hi plane, lo plane),
// rows of Ls >= L tokens.  Y is written as a bf16 pair.
chela_status_t launch_gemm_sm100_at(const void *at, int B, int L, int Ls, const void *w, const float *bias, void *y, int K, int N,
                                    int act, int *status, cudaStream_t stream)
{
    const size_t M = (size_t)B * L;
    const __nv_bfloat16 *a_hi = (const __nv_bfloat16 *)at, *a_lo = a_hi + (size_t)B * K * Ls;
    __nv_bfloat16 *y_hi = (__nv_bfloat16 *)y, *y_lo = y_hi + M * N;
    CUtensorMap ma_hi, ma_lo, mw, my_hi, my_lo;
    const cuuint64_t dims[3] = {(cuuint64_t)L, (cuuint64_t)K, (cuuint64_t)B};
    const cuuint64_t strides[2] = {(cuuint64_t)Ls * 2, (cuuint64_t)K * Ls * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)BK, 1};
    if (!make_map_sw128(&ma_hi, a_hi, false, 3, dims, strides, box) || !make_map_sw128(&ma_lo, a_lo, false, 3, dims, strides, box) ||
        !map_2d(&mw, w, K, N, 64, BK) || !map_2d(&my_hi, y_hi, M, N, 64, 32) || !map_2d(&my_lo, y_lo, M, N, 64, 32))
        return CHELA_ERR_CUDA;
    int sms = 0, dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        sms = 148;
    const long long tiles = (long long)(M / BM) * (N / 256);
    const int grid = (int)(tiles < sms ? tiles : sms);
    auto kern = gemm_sm100_kernel<256, true, true, true>;
    constexpr int smem = Smem<256, true>::bytes;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return CHELA_ERR_CUDA;
    kern<<<grid, kThreads, smem, stream>>>(ma_hi, ma_lo, mw, my_hi, my_lo, bias, (int)M, N, K, act, status, L, current_wait_ctl());
    return last_launch_status();
}

}  // namespace chela
