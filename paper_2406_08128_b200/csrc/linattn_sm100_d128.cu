// Chunked causal linear attention on sm_100a for head dimension 128 (d_k = d_v = 128): the same
// tcgen05 / TMEM / TMA scheme as the 64-wide kernel, with N = 128 instructions (64 cycles each, the
// tensor core's full rate) wherever d_v is the N dimension.
//
// One CTA (issuer warp + 4 compute warps) walks one (batch, head) sequence in tiles of 64 tokens.  Per tile
// and per input plane the TMA ring holds six [64 rows] x 128 B tiles: Q_a, K_a, Q_b, K_b (the two halves of
// d_k, Q and K of a half adjacent) and V_a, V_b (the two halves of d_v, adjacent).
//   G1 : PT   = [Q_a;K_a] Q_a^T + [Q_b;K_b] Q_b^T         rows 64..127 = P^T = K Q^T           (N = 64)
//   G2 : OS_a rows 0..63 = sum_x [Q_x;K_x] (S_x,hi + S_x,lo)   lanes 64..127 write-disabled     (N = 128)
//   G3 : OS_a += [P^T | K_a]^T [V_a|V_b]   rows 0..63 += P V, rows 64..127 += K_a^T V (state rows d_k < 64)
//        S_b  += [P^T | K_b]^T [V_a|V_b]   lanes 0..63 write-disabled: state rows d_k >= 64      (N = 128)
// TMEM: OS_a 128 columns, S_b 128 columns, PT 64 columns.  The fp32 state (128 x 128) never leaves the SM;
// it is fed back as bf16 hi + lo tiles.  With bf16-pair inputs every product takes three terms
// (hi*hi + hi*lo + lo*hi) and the score tile is kept as a pair (the mixer's fp32-like path).
// Sequences are not split along L here (one CTA per (batch, head)).
// Every wait is bounded; a timeout records CHELA_ERR_TIMEOUT, drains outstanding loads, frees TMEM.
#include "sm100_ptx.cuh"

namespace chela {
namespace {

using namespace sm100;

constexpr int kD = 128;
constexpr int kC = 64;
constexpr int kThreads = 160;
constexpr int kTile = kC * 128;

template <typename TOut, bool kPair>
struct Smem {
    static constexpr int kStages = kPair ? 1 : 2;
    static constexpr int kPlanes = kPair ? 2 : 1;
    static constexpr int kOBoxes = (int)sizeof(TOut) * kD / 128;
    static constexpr int offPT = 0;                                   // score tile (hi, lo)
    static constexpr int offS = offPT + kPlanes * kTile;              // S_a hi, S_b hi, S_a lo, S_b lo: 2 tiles each
    static constexpr int offO = offS + 8 * kTile;
    static constexpr int offStage = offO + kOBoxes * kTile;           // per stage and plane: Qa Ka Qb Kb Va Vb
    static constexpr int offBar = offStage + kStages * kPlanes * 6 * kTile;   // full[kStages], p, o, pt, s
    static constexpr int offTmem = offBar + 8 * (kStages + 4);
    static constexpr int offAbort = offTmem + 8;
    static constexpr int bytes = offAbort + 8;
};
constexpr int kTmemCols = 512;
constexpr int kColOS = 0, kColSb = 128, kColPT = 256;

// kReverse: the anti-causal mirror used by the backward pass (chunks walked from the end, upper-triangular mask).
template <typename TOut, bool kPair, bool kReverse>
__global__ void __launch_bounds__(kThreads)
linattn_sm100_d128_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                          const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o, int H, int L,
                          float scale, int norm, float eps, int *__restrict__ status, const float *__restrict__ s_part, int G,
                          int cg0, int cg, const float *__restrict__ state_in, float *__restrict__ state_out)
{
    // Grid: one CTA per (group, batch*head), group-major; group 0 covers the first cg0 chunks, group g >= 1 the next
    // cg each, and starts from state_in[bh] + sum_{g' < g} s_part[bh][g'] (128 x 128 fp32 each); the last group
    // writes state_out[bh].  With G > 1 the kernel is a programmatic dependent of the state kernel: group 0 runs
    // beside it, the others wait for it before reading s_part.
    using SM = Smem<TOut, kPair>;
    constexpr int kStages = SM::kStages, kPlanes = SM::kPlanes;
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    if (sbase & 1023u) {
        if (threadIdx.x == 0) atomicExch(status, (int)CHELA_ERR_CUDA);
        return;
    }
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nbh = gridDim.x / G;
    const int bh = blockIdx.x % nbh, g = blockIdx.x / nbh;
    const int b = bh / H, h = bh % H;
    const int c0 = g == 0 ? 0 : cg0 + (g - 1) * cg;
    const int nch_total = (L + kC - 1) / kC;
    const int nchunks = min(g == 0 ? cg0 : cg, nch_total - c0);
    const bool has_init = g > 0 || state_in != nullptr;
    auto tok = [&](int chunk) { return (kReverse ? nch_total - 1 - (c0 + chunk) : c0 + chunk) * kC; };

    const uint32_t bar_full0 = sbase + SM::offBar;
    const uint32_t bar_p = bar_full0 + 8 * kStages, bar_o = bar_p + 8, bar_pt = bar_o + 8, bar_s = bar_pt + 8;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + SM::offTmem);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + SM::offAbort);

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(bar_full0 + 8 * s, 1);
        mbar_init(bar_p, 1);
        mbar_init(bar_o, 1);
        mbar_init(bar_pt, 2);
        mbar_init(bar_s, 4);
        *abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
        tma_prefetch_desc(&tm_o);
    }
    if (warp == 0) {
        tmem_alloc(sbase + SM::offTmem, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 4) {
        if (lane == 0) {
            // tile t (0 Qa, 1 Ka, 2 Qb, 3 Kb, 4 Va, 5 Vb) of plane pl of the stage of `chunk`
            auto tile = [&](int chunk, int pl, int t) {
                return sbase + SM::offStage + (((chunk % kStages) * kPlanes + pl) * 6 + t) * kTile;
            };
            auto issue_load = [&](int chunk) {
                const uint32_t bar = bar_full0 + 8 * (chunk % kStages);
                mbar_expect_tx(bar, kPlanes * 6 * kTile);
#pragma unroll
                for (int pl = 0; pl < kPlanes; ++pl)
#pragma unroll
                    for (int x = 0; x < 2; ++x) {
                        tma_load_5d(tile(chunk, pl, 2 * x), &tm_q, bar, 64 * x, h, tok(chunk), b, pl);
                        tma_load_5d(tile(chunk, pl, 2 * x + 1), &tm_k, bar, 64 * x, h, tok(chunk), b, pl);
                        tma_load_5d(tile(chunk, pl, 4 + x), &tm_v, bar, 64 * x, h, tok(chunk), b, pl);
                    }
            };
            constexpr uint32_t idescG1 = make_idesc(128, kC, 0, 0);
            constexpr uint32_t idescG2 = make_idesc(128, 128, 0, 1);
            constexpr uint32_t idescG3 = make_idesc(128, 128, 1, 1);
            // G1; false if the chunk's tiles never arrived
            auto issue_scores = [&](int chunk) -> bool {
                if (!mbar_wait(bar_full0 + 8 * (chunk % kStages), (chunk / kStages) & 1, abort_flag)) return false;
                tc_fence_after();
                uint32_t acc = 0;
#pragma unroll
                for (int x = 0; x < 2; ++x) {
                    const uint32_t qk_hi = desc_lo(tile(chunk, 0, 2 * x));
#pragma unroll
                    for (int k = 0; k < 4; ++k) { umma_bf16(tmem + kColPT, qk_hi + 2 * k, qk_hi + 2 * k, idescG1, acc); acc = 1; }
                    if (kPair) {
                        const uint32_t qk_lo = desc_lo(tile(chunk, 1, 2 * x));
#pragma unroll
                        for (int k = 0; k < 4; ++k) umma_bf16(tmem + kColPT, qk_hi + 2 * k, qk_lo + 2 * k, idescG1, 1);
#pragma unroll
                        for (int k = 0; k < 4; ++k) umma_bf16(tmem + kColPT, qk_lo + 2 * k, qk_hi + 2 * k, idescG1, 1);
                    }
                }
                umma_commit(bar_p);
                return true;
            };
            int loads_issued = 0, consumed = 0;
            for (; loads_issued < kStages && loads_issued < nchunks; ++loads_issued) issue_load(loads_issued);
            bool ok = issue_scores(0);
            uint32_t par_s = 0;
            for (int i = 0; ok && i < nchunks; ++i) {
                if (i > 0 || has_init) {
                    ok = mbar_wait(bar_s, par_s, abort_flag);
                    par_s ^= 1;
                    if (!ok) break;
                    tc_fence_after();
                    uint32_t acc = 0;
#pragma unroll
                    for (int x = 0; x < 2; ++x) {
                        // state tiles of d_k half x: hi at offS + x*2 tiles, lo at offS + (4 + x*2) tiles; two d_v atoms each
                        const uint32_t s_hi = desc_lo(sbase + SM::offS + (2 * x) * kTile, kTile),
                                       s_lo = desc_lo(sbase + SM::offS + (4 + 2 * x) * kTile, kTile);
                        const uint32_t qk_hi = desc_lo(tile(i, 0, 2 * x));
#pragma unroll
                        for (int k = 0; k < 4; ++k) { umma_bf16(tmem + kColOS, qk_hi + 2 * k, s_hi + 128 * k, idescG2, acc, 1); acc = 1; }
#pragma unroll
                        for (int k = 0; k < 4; ++k) umma_bf16(tmem + kColOS, qk_hi + 2 * k, s_lo + 128 * k, idescG2, 1, 1);
                        if (kPair) {
                            const uint32_t qk_lo = desc_lo(tile(i, 1, 2 * x));
#pragma unroll
                            for (int k = 0; k < 4; ++k) umma_bf16(tmem + kColOS, qk_lo + 2 * k, s_hi + 128 * k, idescG2, 1, 1);
                        }
                    }
                }
                ok = mbar_wait(bar_pt, i & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                {
                    const uint32_t pt_hi = sbase + SM::offPT, pt_lo = pt_hi + kTile;
                    const uint32_t v_hi = desc_lo(tile(i, 0, 4), kTile);
                    // OS_a: [P^T | K_a] (output rows in lanes 0..63, state rows d_k < 64 in lanes 64..127); S_b: [K_b | next tile]
                    // with the upper lanes write-disabled: state rows d_k >= 64 in lanes 0..63, so that the output warps
                    // convert that half of the state while the score warps convert the other
                    const uint32_t a_a = desc_lo(pt_hi, tile(i, 0, 1) - pt_hi), a_b = desc_lo(tile(i, 0, 3), kTile);
                    const uint32_t first = (i > 0 || has_init) ? 1u : 0u;
#pragma unroll
                    for (int k = 0; k < 4; ++k) umma_bf16(tmem + kColOS, a_a + 128 * k, v_hi + 128 * k, idescG3, (first || k > 0) ? 1u : 0u);
#pragma unroll
                    for (int k = 0; k < 4; ++k) umma_bf16(tmem + kColSb, a_b + 128 * k, v_hi + 128 * k, idescG3, (first || k > 0) ? 1u : 0u, 1);
                    if (kPair) {
                        const uint32_t v_lo = desc_lo(tile(i, 1, 4), kTile);
                        const uint32_t a2_a = desc_lo(pt_lo, tile(i, 1, 1) - pt_lo), a2_b = desc_lo(tile(i, 1, 3), kTile);
#pragma unroll
                        for (int k = 0; k < 4; ++k) umma_bf16(tmem + kColOS, a_a + 128 * k, v_lo + 128 * k, idescG3, 1);
#pragma unroll
                        for (int k = 0; k < 4; ++k) umma_bf16(tmem + kColOS, a2_a + 128 * k, v_hi + 128 * k, idescG3, 1);
#pragma unroll
                        for (int k = 0; k < 4; ++k) umma_bf16(tmem + kColSb, a_b + 128 * k, v_lo + 128 * k, idescG3, 1, 1);
#pragma unroll
                        for (int k = 0; k < 4; ++k) umma_bf16(tmem + kColSb, a2_b + 128 * k, v_hi + 128 * k, idescG3, 1, 1);
                    }
                    umma_commit(bar_o);
                }
                if (kStages > 1 && i + 1 < nchunks) {
                    ok = issue_scores(i + 1);
                    if (!ok) break;
                }
                ok = mbar_wait(bar_o, i & 1, abort_flag);
                if (!ok) break;
                consumed = i + 1;
                if (i + kStages < nchunks) {
                    issue_load(i + kStages);
                    ++loads_issued;
                }
                if (kStages == 1 && i + 1 < nchunks) {
                    ok = issue_scores(i + 1);
                    if (!ok) break;
                }
            }
            if (!ok) {
                *abort_flag = 1;
                atomicExch(status, (int)CHELA_ERR_TIMEOUT);
                for (int c = consumed; c < loads_issued; ++c)
                    mbar_wait(bar_full0 + 8 * (c % kStages), (c / kStages) & 1, nullptr);
            }
        }
    } else {
        const bool upper = warp >= 2;
        const int r = tid & 63;
        const uint32_t tmem_warp = tmem + ((uint32_t)(warp * 32) << 16);
        bool ok = true;
        // state rows of this thread: d_k = r (accumulator OS_a) and d_k = 64 + r (accumulator S_b); hi/lo tiles per
        // d_v half: tile index 2*x + half, low part four tiles later
        auto write_state_tiles = [&](const float(&sv)[64], int x, int half) {
            uint8_t *sHi = smem + SM::offS + (2 * x + half) * kTile, *sLo = sHi + 4 * kTile;
#pragma unroll
            for (int c8 = 0; c8 < 8; ++c8) {
                uint32_t wh[4], wl[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float x0 = sv[c8 * 8 + e * 2], x1 = sv[c8 * 8 + e * 2 + 1];
                    const __nv_bfloat162 hh = __floats2bfloat162_rn(x0, x1);
                    const float2 hf = __bfloat1622float2(hh);
                    float l0, l1;
                    sub2(l0, l1, x0, x1, hf.x, hf.y);
                    wh[e] = *reinterpret_cast<const uint32_t *>(&hh);
                    wl[e] = pack_bf16(l0, l1);
                }
                const uint32_t off = sw128(r, c8);
                *reinterpret_cast<uint4 *>(sHi + off) = make_uint4(wh[0], wh[1], wh[2], wh[3]);
                *reinterpret_cast<uint4 *>(sLo + off) = make_uint4(wl[0], wl[1], wl[2], wl[3]);
            }
        };
        // state rows of this thread: d_k = 64 * xs + r, xs = 0 for the score warps (accumulator OS_a, lanes 64..127), 1 for the
        // output warps (accumulator S_b, lanes 0..63)
        const int xs = upper ? 0 : 1;
        if (has_init) {
            {
                const int x = xs;
#pragma unroll 1
                    for (int half = 0; half < 2; ++half) {
                        float sv[64];
#pragma unroll
                        for (int j = 0; j < 64; ++j) sv[j] = 0.f;
                        const size_t row_off = (size_t)(64 * x + r) * kD + 64 * half;
                        auto add_row = [&](const float *base) {
                            const float4 *src = reinterpret_cast<const float4 *>(base + row_off);
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const float4 t = src[j];
                                sv[4 * j] += t.x; sv[4 * j + 1] += t.y; sv[4 * j + 2] += t.z; sv[4 * j + 3] += t.w;
                            }
                        };
                        if (state_in) add_row(state_in + (size_t)bh * kD * kD);
                        if (g > 0) griddep_wait();   // the state kernel has completed
                        for (int gp = 0; gp < g; ++gp) add_row(s_part + ((size_t)bh * (G - 1) + gp) * kD * kD);
                        const uint32_t col = (x == 0 ? kColOS : kColSb) + 64 * half;
                        tmem_st32(tmem_warp + col, *reinterpret_cast<const float(*)[32]>(&sv[0]));
                        tmem_st32(tmem_warp + col + 32, *reinterpret_cast<const float(*)[32]>(&sv[32]));
                        tmem_st_wait();
                        write_state_tiles(sv, x, half);
                    }
                fence_proxy_async();
                tc_fence_before();
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_s);
        }
        for (int i = 0; i < nchunks; ++i) {
            if (upper) {
                // ---- P^T_i: TMEM -> causal mask (t >= s) -> bf16 (pair) -> shared, rows = s ---------------
                ok = __all_sync(0xffffffffu, mbar_wait(bar_p, i & 1, abort_flag));
                if (!ok) break;
                tc_fence_after();
                float p[2][32];
                const bool live0 = kReverse || warp == 2, live1 = !kReverse || warp == 3;
                if (live0) tmem_ld32(tmem_warp + kColPT, p[0]);
                if (live1) tmem_ld32(tmem_warp + kColPT + 32, p[1]);
                tmem_ld_wait();
                uint8_t *sP = smem + SM::offPT;
#pragma unroll
                for (int cb = 0; cb < 2; ++cb) {
                    const bool live = cb == 0 ? live0 : live1;
#pragma unroll
                    for (int c8 = 0; c8 < 4; ++c8) {
                        uint32_t w[4], w2[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int t = cb * 32 + c8 * 8 + e * 2;
                            const float x0 = (live && (kReverse ? t <= r : t >= r)) ? p[cb][c8 * 8 + e * 2] : 0.f;
                            const float x1 = (live && (kReverse ? t + 1 <= r : t + 1 >= r)) ? p[cb][c8 * 8 + e * 2 + 1] : 0.f;
                            const __nv_bfloat162 hh = __floats2bfloat162_rn(x0, x1);
                            w[e] = *reinterpret_cast<const uint32_t *>(&hh);
                            if (kPair) {
                                const float2 hf = __bfloat1622float2(hh);
                                w2[e] = pack_bf16(x0 - hf.x, x1 - hf.y);
                            }
                        }
                        *reinterpret_cast<uint4 *>(sP + sw128(r, cb * 4 + c8)) = make_uint4(w[0], w[1], w[2], w[3]);
                        if (kPair) *reinterpret_cast<uint4 *>(sP + kTile + sw128(r, cb * 4 + c8)) = make_uint4(w2[0], w2[1], w2[2], w2[3]);
                    }
                }
                fence_proxy_async();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_pt);
            }
            ok = __all_sync(0xffffffffu, mbar_wait(bar_o, i & 1, abort_flag));
            if (!ok) break;
            tc_fence_after();
            // ---- state rows d_k = 64 * xs + r of this thread: bf16 hi + lo -> shared (B operand of the next chunk's G2) ----
            auto convert_state_rows = [&]() {
#pragma unroll 1
                for (int half = 0; half < 2; ++half) {
                    float sv[64];
                    const uint32_t col = (xs == 0 ? kColOS : kColSb) + 64 * half;
                    tmem_ld32(tmem_warp + col, *reinterpret_cast<float(*)[32]>(&sv[0]));
                    tmem_ld32(tmem_warp + col + 32, *reinterpret_cast<float(*)[32]>(&sv[32]));
                    tmem_ld_wait();
                    write_state_tiles(sv, xs, half);
                }
                fence_proxy_async();
            };
            // last chunk of the sequence: the fp32 state leaves the SM once, for the caller
            auto store_state_rows = [&]() {
#pragma unroll 1
                for (int half = 0; half < 2; ++half) {
                    float sv[64];
                    const uint32_t col = (xs == 0 ? kColOS : kColSb) + 64 * half;
                    tmem_ld32(tmem_warp + col, *reinterpret_cast<float(*)[32]>(&sv[0]));
                    tmem_ld32(tmem_warp + col + 32, *reinterpret_cast<float(*)[32]>(&sv[32]));
                    tmem_ld_wait();
                    float4 *dst = reinterpret_cast<float4 *>(state_out + (size_t)bh * kD * kD + (size_t)(64 * xs + r) * kD + 64 * half);
#pragma unroll
                    for (int j = 0; j < 16; ++j) dst[j] = make_float4(sv[4 * j], sv[4 * j + 1], sv[4 * j + 2], sv[4 * j + 3]);
                }
            };
            if (!upper) {
                // their half of the state first (the next chunk's G2 waits for it), then the output rows
                if (i + 1 < nchunks) convert_state_rows();
                else if (state_out && g == G - 1) store_state_rows();
                // ---- output row t (128 values): scale, normaliser -> swizzled staging -> TMA store ------------
                float acc[kD];
#pragma unroll
                for (int c = 0; c < 4; ++c) tmem_ld32(tmem_warp + kColOS + 32 * c, *reinterpret_cast<float(*)[32]>(&acc[32 * c]));
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(bar_s);
                    bulk_wait_read0();
                }
                __syncwarp();
                float ss = 0.f;
#pragma unroll
                for (int j = 0; j < kD; ++j) {
                    acc[j] *= scale;
                    ss = fmaf(acc[j], acc[j], ss);
                }
                const float inv = norm ? rsqrtf(ss * (1.0f / kD) + eps) : 1.0f;
                uint8_t *sO = smem + SM::offO;
                if (sizeof(TOut) == 4) {
#pragma unroll
                    for (int j = 0; j < kD; j += 4)
                        *reinterpret_cast<float4 *>(sO + (j / 32) * kTile + sw128(r, (j % 32) / 4)) =
                            make_float4(acc[j] * inv, acc[j + 1] * inv, acc[j + 2] * inv, acc[j + 3] * inv);
                } else {
#pragma unroll
                    for (int j = 0; j < kD; j += 8)
                        *reinterpret_cast<uint4 *>(sO + (j / 64) * kTile + sw128(r, (j % 64) / 8)) =
                            make_uint4(pack_bf16(acc[j] * inv, acc[j + 1] * inv), pack_bf16(acc[j + 2] * inv, acc[j + 3] * inv),
                                       pack_bf16(acc[j + 4] * inv, acc[j + 5] * inv), pack_bf16(acc[j + 6] * inv, acc[j + 7] * inv));
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
#pragma unroll
                    for (int bx = 0; bx < SM::kOBoxes; ++bx)
                        tma_store_5d(&tm_o, sbase + SM::offO + bx * kTile + warp * 32 * 128, bx * (128 / (int)sizeof(TOut)), h,
                                     tok(i) + warp * 32, b, 0);
                    bulk_commit();
                }
            } else if (i + 1 < nchunks) {
                convert_state_rows();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_s);
            } else if (state_out && g == G - 1) {
                store_state_rows();
            }
        }
        if (!ok && lane == 0) {
            *abort_flag = 1;
            atomicExch(status, (int)CHELA_ERR_TIMEOUT);
        }
        if (!upper && lane == 0) bulk_wait0();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// Per-group state sums for sequences split along L: CTA (batch*head, g), g < G-1, writes
// s_part[bh][g] = sum over the group's chunks of K_i^T V_i (128 x 128 fp32).  One accumulator, M = N = 128:
// A = [K_a | K_b] (MN-major, the two d_k halves are adjacent tiles), B = [V_a | V_b].
template <bool kPair>
struct SmemState {
    static constexpr int kStages = kPair ? 2 : 3;
    static constexpr int kPlanes = kPair ? 2 : 1;
    static constexpr int offStage = 0;                                        // per stage and plane: Ka Kb Va Vb
    static constexpr int offBar = kStages * kPlanes * 4 * kTile;              // full[], empty[], done
    static constexpr int offTmem = offBar + 8 * (2 * kStages + 1);
    static constexpr int offAbort = offTmem + 8;
    static constexpr int bytes = offAbort + 8;
};

template <bool kPair, bool kReverse>
__global__ void __launch_bounds__(kThreads)
linattn_state_d128_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                          float *__restrict__ s_part, int H, int L, int G, int cg0, int cg, int *__restrict__ status)
{
    using SM = SmemState<kPair>;
    constexpr int kStages = SM::kStages, kPlanes = SM::kPlanes;
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    if (sbase & 1023u) {
        if (threadIdx.x == 0) atomicExch(status, (int)CHELA_ERR_CUDA);
        return;
    }
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    griddep_launch_dependents();   // the main kernel's first groups may be scheduled beside this kernel
    const int nbh = gridDim.x / (G - 1);
    const int bh = blockIdx.x % nbh, g = blockIdx.x / nbh;
    const int b = bh / H, h = bh % H;
    const int c0 = g == 0 ? 0 : cg0 + (g - 1) * cg, nchunks = g == 0 ? cg0 : cg;
    const uint32_t bar_full0 = sbase + SM::offBar, bar_empty0 = bar_full0 + 8 * kStages, bar_done = bar_empty0 + 8 * kStages;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + SM::offTmem);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + SM::offAbort);
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar_full0 + 8 * s, 1);
            mbar_init(bar_empty0 + 8 * s, 1);
        }
        mbar_init(bar_done, 1);
        *abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
    }
    if (warp == 0) {
        tmem_alloc(sbase + SM::offTmem, 128);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 4) {
        if (lane == 0) {
            auto tile = [&](int chunk, int pl, int t) { return sbase + SM::offStage + (((chunk % kStages) * kPlanes + pl) * 4 + t) * kTile; };
            auto issue_load = [&](int chunk) {
                const uint32_t bar = bar_full0 + 8 * (chunk % kStages);
                mbar_expect_tx(bar, kPlanes * 4 * kTile);
#pragma unroll
                for (int pl = 0; pl < kPlanes; ++pl)
#pragma unroll
                    for (int x = 0; x < 2; ++x) {
                        const int t0 = (kReverse ? (L + kC - 1) / kC - 1 - (c0 + chunk) : c0 + chunk) * kC;
                        tma_load_5d(tile(chunk, pl, x), &tm_k, bar, 64 * x, h, t0, b, pl);
                        tma_load_5d(tile(chunk, pl, 2 + x), &tm_v, bar, 64 * x, h, t0, b, pl);
                    }
            };
            constexpr uint32_t idesc = make_idesc(128, 128, 1, 1);
            int loads_issued = 0, consumed = 0;
            for (; loads_issued < kStages && loads_issued < nchunks; ++loads_issued) issue_load(loads_issued);
            bool ok = true;
            for (int i = 0; i < nchunks; ++i) {
                const int stage = i % kStages;
                ok = mbar_wait(bar_full0 + 8 * stage, (i / kStages) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t k_hi = desc_lo(tile(i, 0, 0), kTile), v_hi = desc_lo(tile(i, 0, 2), kTile);
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_bf16(tmem, k_hi + 128 * k, v_hi + 128 * k, idesc, (i > 0 || k > 0) ? 1u : 0u);
                if (kPair) {
                    const uint32_t k_lo = desc_lo(tile(i, 1, 0), kTile), v_lo = desc_lo(tile(i, 1, 2), kTile);
#pragma unroll
                    for (int k = 0; k < 4; ++k) umma_bf16(tmem, k_hi + 128 * k, v_lo + 128 * k, idesc, 1);
#pragma unroll
                    for (int k = 0; k < 4; ++k) umma_bf16(tmem, k_lo + 128 * k, v_hi + 128 * k, idesc, 1);
                }
                umma_commit(bar_empty0 + 8 * stage);
                consumed = i + 1;
                if (i + kStages < nchunks) {
                    ok = mbar_wait(bar_empty0 + 8 * stage, (i / kStages) & 1, abort_flag);
                    if (!ok) break;
                    issue_load(i + kStages);
                    ++loads_issued;
                }
            }
            if (ok) umma_commit(bar_done);
            else {
                *abort_flag = 1;
                atomicExch(status, (int)CHELA_ERR_TIMEOUT);
                for (int c = consumed; c < loads_issued; ++c) mbar_wait(bar_full0 + 8 * (c % kStages), (c / kStages) & 1, nullptr);
            }
        }
    } else {
        const bool ok = __all_sync(0xffffffffu, mbar_wait(bar_done, 0, abort_flag));
        if (ok) {
            tc_fence_after();
            const uint32_t tmem_warp = tmem + ((uint32_t)(warp * 32) << 16);
            float4 *dst = reinterpret_cast<float4 *>(s_part + (((size_t)bh * (G - 1) + g) * kD + tid) * kD);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                float sv[64];
                tmem_ld32(tmem_warp + 64 * half, *reinterpret_cast<float(*)[32]>(&sv[0]));
                tmem_ld32(tmem_warp + 64 * half + 32, *reinterpret_cast<float(*)[32]>(&sv[32]));
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 16; ++j) dst[16 * half + j] = make_float4(sv[4 * j], sv[4 * j + 1], sv[4 * j + 2], sv[4 * j + 3]);
            }
        } else if (lane == 0) {
            *abort_flag = 1;
            atomicExch(status, (int)CHELA_ERR_TIMEOUT);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 128);
}

bool make_map(CUtensorMap *map, const void *ptr, int B, int H, int L, int box_rows, bool f32, int planes)
{
    const cuuint64_t es = f32 ? 4 : 2;
    const cuuint64_t dims[5] = {(cuuint64_t)kD, (cuuint64_t)H, (cuuint64_t)L, (cuuint64_t)B, (cuuint64_t)planes};
    const cuuint64_t strides[4] = {(cuuint64_t)kD * es, (cuuint64_t)H * kD * es, (cuuint64_t)L * H * kD * es,
                                   (cuuint64_t)B * L * H * kD * es};
    const cuuint32_t box[5] = {(cuuint32_t)(128 / es), 1, (cuuint32_t)box_rows, 1, 1};
    return make_map_sw128(map, ptr, f32, 5, dims, strides, box);
}

// Split along L: one CTA per SM is resident (shared memory), at least 16 chunks per group.
struct SplitPlan {
    int G, cg0, cg;   // group 0: cg0 chunks, the others cg (two groups: the first a quarter longer, it runs beside the state kernel)
    size_t part_bytes;
};
SplitPlan split_plan(int B, int H, int L, int sms = 0)
{
    int dev = 0;
    if (sms <= 0 && (cudaGetDevice(&dev) != cudaSuccess ||
                     cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0))
        sms = 148;
    const long long bh = (long long)B * H;
    const int nchunks = (L + kC - 1) / kC;
    int G = 1;
    if (bh * 2 <= sms) {
        G = (int)(sms / bh);
        if (G > nchunks / 16) G = nchunks / 16;
        if (G < 1) G = 1;
    }
    SplitPlan p;
    if (G == 1) {
        p.G = 1;
        p.cg0 = p.cg = nchunks;
    } else {
        const double rho = G == 2 ? 0.8 : 1.0;   // measured: one CTA per SM, the state pass costs 0.23 of the main pass per chunk
        p.cg0 = (int)((double)nchunks / (1.0 + (G - 1) * rho) + 0.999);
        if (p.cg0 > nchunks - (G - 1)) p.cg0 = nchunks - (G - 1);
        p.cg = (nchunks - p.cg0 + G - 2) / (G - 1);
        p.G = 1 + (nchunks - p.cg0 + p.cg - 1) / p.cg;
    }
    p.part_bytes = (size_t)bh * (p.G - 1) * kD * kD * sizeof(float);
    return p;
}
constexpr size_t kWsHeader = 512;

template <typename TOut, bool kPair, bool kReverse>
chela_status_t launch_t(const void *q, const void *k, const void *v, void *o, int B, int H, int L, int norm, float eps,
                        float scale, void *workspace, const float *state_in, float *state_out, cudaStream_t stream,
                        int pair_mask = 7, bool keep_status = false)
{
    // pair_mask: which of q, k, v really are pairs; a single bf16 operand of a pair kernel gets a one-plane map
    // and its low plane arrives as zeros (out of bounds for the copy engine)
    CUtensorMap mq, mk, mv, mo;
    const int pq = (kPair && (pair_mask & 1)) ? 2 : 1, pk = (kPair && (pair_mask & 2)) ? 2 : 1, pv = (kPair && (pair_mask & 4)) ? 2 : 1;
    if (!make_map(&mq, q, B, H, L, kC, false, pq) || !make_map(&mk, k, B, H, L, kC, false, pk) ||
        !make_map(&mv, v, B, H, L, kC, false, pv) || !make_map(&mo, o, B, H, L, 32, sizeof(TOut) == 4, 1))
        return CHELA_ERR_CUDA;
    int *status = (int *)workspace;
    float *s_part = (float *)((char *)workspace + kWsHeader);
    const SplitPlan plan = split_plan(B, H, L);
    if (!keep_status && cudaMemsetAsync(status, 0, sizeof(int), stream) != cudaSuccess) return CHELA_ERR_CUDA;
    if (plan.G > 1) {
        auto skern = linattn_state_d128_kernel<kPair, kReverse>;
        if (cudaFuncSetAttribute(skern, cudaFuncAttributeMaxDynamicSharedMemorySize, SmemState<kPair>::bytes) != cudaSuccess)
            return CHELA_ERR_CUDA;
        skern<<<B * H * (plan.G - 1), kThreads, SmemState<kPair>::bytes, stream>>>(mk, mv, s_part, H, L, plan.G, plan.cg0, plan.cg, status);
        if (cudaGetLastError() != cudaSuccess) return CHELA_ERR_CUDA;
    }
    auto kern = linattn_sm100_d128_kernel<TOut, kPair, kReverse>;
    const int smem = Smem<TOut, kPair>::bytes;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return CHELA_ERR_CUDA;
    if (plan.G > 1) {   // may start while the state kernel still runs
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(B * H * plan.G);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, kern, mq, mk, mv, mo, H, L, scale, norm, eps, status, (const float *)s_part, plan.G, plan.cg0,
                               plan.cg, state_in, state_out) != cudaSuccess) {
            // without the attribute: an ordinary stream-ordered launch (griddepcontrol.wait returns at once)
            (void)cudaGetLastError();
            kern<<<B * H * plan.G, kThreads, smem, stream>>>(mq, mk, mv, mo, H, L, scale, norm, eps, status, s_part, plan.G, plan.cg0,
                                                             plan.cg, state_in, state_out);
        }
        return last_launch_status();
    }
    kern<<<B * H, kThreads, smem, stream>>>(mq, mk, mv, mo, H, L, scale, norm, eps, status, s_part, 1, plan.cg0, plan.cg, state_in,
                                            state_out);
    return last_launch_status();
}

}  // namespace

size_t linattn_sm100_d128_workspace_bytes(int B, int H, int L) { return kWsHeader + split_plan(B, H, L).part_bytes; }

void linattn_sm100_d128_split(int B, int H, int L, int sms, int *G, int *cg0, int *cg)
{
    const SplitPlan p = split_plan(B, H, L, sms);
    *G = p.G;
    *cg0 = p.cg0;
    *cg = p.cg;
}

chela_status_t launch_linattn_sm100_d128(const void *q, const void *k, const void *v, void *o, int B, int H, int L,
                                         chela_dtype_t in_dtype, chela_dtype_t out_dtype, int norm, float eps, float scale,
                                         void *workspace, cudaStream_t stream, const float *state_in, float *state_out, bool reverse,
                                         int pair_mask, bool keep_status)
{
    if (reverse) {
        if (out_dtype != CHELA_F32 || state_in || state_out) return CHELA_ERR_UNSUPPORTED;
        if (in_dtype == CHELA_BF16_PAIR)
            return launch_t<float, true, true>(q, k, v, o, B, H, L, norm, eps, scale, workspace, nullptr, nullptr, stream, pair_mask, keep_status);
        return launch_t<float, false, true>(q, k, v, o, B, H, L, norm, eps, scale, workspace, nullptr, nullptr, stream, 7, keep_status);
    }
    if (in_dtype == CHELA_BF16_PAIR) {
        if (out_dtype == CHELA_F32)
            return launch_t<float, true, false>(q, k, v, o, B, H, L, norm, eps, scale, workspace, state_in, state_out, stream, pair_mask, keep_status);
        return launch_t<__nv_bfloat16, true, false>(q, k, v, o, B, H, L, norm, eps, scale, workspace, state_in, state_out, stream, 7, keep_status);
    }
    if (out_dtype == CHELA_F32) return launch_t<float, false, false>(q, k, v, o, B, H, L, norm, eps, scale, workspace, state_in, state_out, stream, 7, keep_status);
    return launch_t<__nv_bfloat16, false, false>(q, k, v, o, B, H, L, norm, eps, scale, workspace, state_in, state_out, stream, 7, keep_status);
}

}  // namespace chela
